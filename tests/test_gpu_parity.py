"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle on the same inputs.

Tolerances (relative Frobenius error against the oracle): 1e-5 on the fp32 CUDA-core path,
2e-3 on the TF32 path, 1e-2 on the bf16-in / fp32-accumulate path; SF buffer layout, indices and
pure copies bit-exact.
"""
import numpy as np
import pytest
import torch

from oracle import sfb_oracle as orc
from sfbgen import get_config, make_inputs, scaled
from tests.util import (MAX_STORAGE_OVER_TOL, MODEL_ID, TOL, assert_lines, batch_of, dml_accept_gate, oracle_apply,
                        oracle_factors, to_f64)

pytestmark = pytest.mark.gpu


def _workload(cfg, inputs, path, guard=False):
    from paper_1511_08486_b200.workload import DeviceWorkload
    return DeviceWorkload(cfg, inputs, path=path, guard=guard)


def _wire_dtype(path):
    return orc.DTYPE_BF16 if path == "bf16" else orc.DTYPE_F32


def _oracle_pack_of(cfg, path, U, V, batch, inputs, clock):
    csr = (batch["rowptr"], batch["idx"], batch["val"]) if cfg["model"] == "sc" else None
    return orc.pack(MODEL_ID[cfg["model"]], _wire_dtype(path), cfg["J"], cfg["D"], cfg["P"], cfg["B"], U, V, csr=csr,
                    clock=clock, nnz_capacity=inputs.get("nnz_capacity", 0))


_ORACLE_MEMO = {}


def _memo(cfg, tag, fn):
    """Oracle results that several tests of one session ask for again (the same workload on another arithmetic
    path): computed once.  Keyed by everything that determines the synthetic inputs and the request."""
    key = (tag,) + tuple(sorted((k, repr(v)) for k, v in cfg.items() if k not in ("path", "compact")))
    if key not in _ORACLE_MEMO:
        if len(_ORACLE_MEMO) > 8:
            _ORACLE_MEMO.clear()
        _ORACLE_MEMO[key] = fn()
    return _ORACLE_MEMO[key]


def _sc_update_from_zero(cfg, U, batch, n_rows=None):
    """U^T A for sparse codes A: the oracle's sparse apply to W = 0 with eta = -1, or, for workloads whose K outer
    products would take its Python loop minutes, the dense product of the same codes (the same sum; the two routes
    are pinned equal on the CPU)."""
    J, D = cfg["J"], cfg["D"]
    n = cfg["K"] if n_rows is None else n_rows
    rp = batch["rowptr"][:n + 1]
    if int(rp[-1]) < 100000:
        return orc.apply_sparse(np.zeros((J, D)), U[:n], rp, batch["idx"], batch["val"], -1.0)
    A = _memo(cfg, "dense codes", lambda: orc.csr_to_dense(batch["rowptr"], batch["idx"], batch["val"], D))
    return orc.delta_w(U[:n], A[:n])


def check_config(cfg, path, eta=None, steps=2, check_v_exact=True, guard=False):
    """guard: W, the SF buffer, U and V sit between guard bands of NaN patterns that must survive every call."""
    inputs = make_inputs(cfg)
    wl = _workload(cfg, inputs, path, guard=guard)
    tol = TOL[path]
    J, D, K = cfg["J"], cfg["D"], cfg["K"]
    eta = cfg["eta"] if eta is None else eta
    W0 = inputs["W"]
    batch = batch_of(inputs, cfg, 0)
    try:
        # ---- factors -----------------------------------------------------------------------------
        U_or, V_or, extra = _memo(cfg, "factors at W0", lambda: oracle_factors(cfg, W0, batch))
        wl.compute_factors(0)
        torch.cuda.synchronize()
        U_gpu = to_f64(wl.U)[:, :J]
        assert not to_f64(wl.U)[:, J:].any(), "pad columns of U must be zero"
        U_ref = dml_accept_gate(cfg, U_gpu, U_or, extra, path) if cfg["model"] == "dml" else U_or
        e_u = orc.rel_fro(U_gpu, U_ref)
        assert e_u <= tol, f"E_U = {e_u:.3e} > {tol}"
        assert_lines(U_gpu, U_ref, tol, "U")                 # no single sample's u, no single class, is far off
        if cfg["model"] != "sc":
            V_gpu = to_f64(wl.V)
            assert not V_gpu[:, D:].any(), "pad columns of V must be zero"
            if check_v_exact:
                assert np.array_equal(V_gpu[:, :D], V_or), "v is a pure copy (MLR) / one fp32 subtraction (DML)"
        # ---- pack: the buffer is exactly the oracle's serialisation of the same (U, V) -----------
        wl.pack(0, clock=5)
        torch.cuda.synchronize()
        buf = wl.sf_buf.cpu().numpy()
        ref_buf = _oracle_pack_of(cfg, path, U_gpu, V_or, batch, inputs, 5)
        assert buf.size == ref_buf.size
        assert np.array_equal(buf, ref_buf), f"SF buffer differs at byte {np.nonzero(buf != ref_buf)[0][:4]}"
        # ---- apply to zero: W = 0, eta = -1 gives U^T V ---------------------------------------------
        wl.W.zero_()
        wl.ctx.invalidate()
        wl.apply(-1.0)
        torch.cuda.synchronize()
        dW_gpu = to_f64(wl.W)
        if cfg["model"] == "sc":
            dW_or = _sc_update_from_zero(cfg, U_gpu, batch)
        else:
            dW_or = orc.delta_w(U_gpu, V_or)
        e_dw = orc.rel_fro(dW_gpu, dW_or)
        assert e_dw <= tol, f"E_dW = {e_dw:.3e} > {tol}"
        assert_lines(dW_gpu, dW_or, tol, "U^T V")            # no row, no column of the update is far off
        # partial apply: only the first worker's stream
        if cfg["P"] > 1:
            wl.W.zero_()
            wl.ctx.invalidate()
            wl.apply(-1.0, K=cfg["B"])
            torch.cuda.synchronize()
            Bn = cfg["B"]
            if cfg["model"] == "sc":
                ref1 = _sc_update_from_zero(cfg, U_gpu, batch, Bn)
            else:
                ref1 = orc.delta_w(U_gpu[:Bn], V_or[:Bn])
            assert orc.rel_fro(to_f64(wl.W), ref1) <= tol
            assert_lines(to_f64(wl.W), ref1, tol, "U^T V of the first worker")
        # ---- steps: W_T - W_0 against the oracle's trajectory ----------------------------------------
        def trajectory():
            W_t = W0.astype(np.float64)
            for t in range(steps):
                bt = batch_of(inputs, cfg, t % cfg["pool"])
                U_t, V_t, _ = oracle_factors(cfg, W_t, bt)
                W_t = oracle_apply(cfg, W_t, U_t, V_t, bt, eta)
            return W_t
        # (DML is checked step by step from the GPU's own state below: no free-running trajectory)
        W_or = None if cfg["model"] == "dml" else _memo(cfg, ("trajectory", float(eta), steps), trajectory)
        runs = []
        for rep in range(2):
            wl.reset()
            for t in range(steps):
                wl.step(t, eta=eta)
            torch.cuda.synchronize()
            runs.append((wl.W.cpu().numpy().copy(), wl.sf_buf.cpu().numpy().copy()))
        assert np.array_equal(runs[0][0], runs[1][0]) and np.array_equal(runs[0][1], runs[1][1]), \
            "two runs from the same state must be bit-identical"
        W_gpu = runs[0][0].astype(np.float64)
        if cfg["model"] == "dml":
            # The hinge gate is discontinuous: a pair within the tie band may legitimately take either
            # value, after which free-running trajectories differ.  So every step is checked on its own,
            # started from the GPU's current L, with the GPU's gate accepted on in-band pairs only.
            wl.reset()
            e_step = 0.0
            for t in range(steps):
                bt = batch_of(inputs, cfg, t % cfg["pool"])
                W_t = wl.W.cpu().numpy()
                wl.step(t, eta=eta)
                torch.cuda.synchronize()
                _, U_wire, _ = orc.unpack(wl.sf_buf.cpu().numpy())
                U_o, V_o, ex = oracle_factors(cfg, W_t, bt)
                U_fix = dml_accept_gate(cfg, U_wire.astype(np.float64), U_o, ex, path)
                ref_move = -eta * orc.delta_w(U_fix, V_o)
                got_move = wl.W.cpu().numpy().astype(np.float64) - W_t.astype(np.float64)
                storage = 2.0 ** -24 * np.linalg.norm(W_t) / np.linalg.norm(ref_move)
                assert storage <= MAX_STORAGE_OVER_TOL * tol, f"storage term {storage:.1e} swamps the tolerance: raise eta"
                e_t = np.linalg.norm(got_move - ref_move) / np.linalg.norm(ref_move)
                assert e_t <= tol + storage, f"step {t}: E_step = {e_t:.3e} > {tol} + {storage:.1e}"
                W_t64 = W_t.astype(np.float64)
                assert_lines(got_move, ref_move, tol, f"step {t}: W' - W",
                             extra_rows=2.0 ** -24 * np.linalg.norm(W_t64, axis=1),
                             extra_cols=2.0 ** -24 * np.linalg.norm(W_t64, axis=0))
                e_step = max(e_step, e_t)
        else:
            moved = np.linalg.norm(W_or - W0)
            e_step = np.linalg.norm((W_gpu - W0) - (W_or - W0)) / moved
            # W is stored in fp32: every step rounds it once (at most 2^-24 relative per element, independent from
            # step to step, so T roundings add up like sqrt(T)); that is not the kernel's error
            storage = np.sqrt(steps) * 2.0 ** -24 * np.linalg.norm(W0) / moved
            assert storage <= MAX_STORAGE_OVER_TOL * tol, f"storage term {storage:.1e} swamps the tolerance: raise eta"
            assert e_step <= tol + storage, f"E_step = {e_step:.3e} > {tol} + {storage:.1e}"
            W064 = W0.astype(np.float64)
            assert_lines(W_gpu - W064, W_or - W064, tol, "W_T - W_0",
                         extra_rows=np.sqrt(steps) * 2.0 ** -24 * np.linalg.norm(W064, axis=1),
                         extra_cols=np.sqrt(steps) * 2.0 ** -24 * np.linalg.norm(W064, axis=0))
        # the buffer left by the last step is a valid serialisation with the step's clock
        h, U_last, _ = orc.unpack(runs[0][1])
        assert h["clock"] == steps - 1 and h["P"] == cfg["P"] and h["J"] == J
        assert wl.ctx.status() == 0
        assert wl.guards_intact(), "a kernel wrote outside W, the SF buffer, U or V"
        return dict(e_u=e_u, e_dw=e_dw, e_step=e_step)
    finally:
        wl.close()


# ------------------------------------------------------------------------------------- fp32 CUDA-core path
def test_c0_mlr_tiny_f32():
    cfg = get_config("C0")
    check_config(cfg, "f32", eta=cfg["eta"], steps=1)
    check_config(cfg, "f32", eta=20.0, steps=3)          # large step: the update dominates fp32 storage rounding


@pytest.mark.parametrize("P,B", [(1, 32), (4, 8), (32, 1)])
def test_c0_worker_split_invariance(P, B):
    cfg = scaled("C0", P=P, B=B)
    cfg["name"] = "C0"
    check_config(cfg, "f32", eta=1.0, steps=1)


def test_mlr_ragged_shapes_f32():
    # J, D, K not multiples of any tile size; D not a multiple of 4 exercises the scalar edges
    for J, D, P, B in ((37, 203, 3, 7), (130, 516, 2, 65), (257, 1000, 5, 13)):
        check_config(scaled("C1", J=J, D=D, P=P, B=B, pool=2), "f32", eta=0.5, steps=2)


def test_c1_mlr_large_scaled_f32():
    check_config(scaled("C1", J=500, D=4000, P=8, B=32, pool=3), "f32", eta=1.0, steps=3)


def test_c1_mlr_large_full_f32():
    check_config(get_config("C1"), "f32", eta=1.0, steps=1)


def test_c2_dml_scaled_f32():
    check_config(scaled("C2", J=72, D=1001, P=3, B=20), "f32", eta=1e-4, steps=2)
    check_config(scaled("C2", J=600, D=2000, P=8, B=32), "f32", eta=1e-4, steps=2)


def test_c2_dml_full_f32():
    check_config(get_config("C2"), "f32", eta=1e-5, steps=1)


def test_c3_sc_scaled_f32():
    check_config(scaled("C3", J=70, D=333, P=3, B=5, density=0.1), "f32", eta=1e-2, steps=2)
    check_config(scaled("C3", J=512, D=2000, P=4, B=32), "f32", eta=1e-3, steps=2)


def test_c3_sc_many_samples_f32():
    """K beyond one shared-memory slice of the scatter apply: two ragged slices, then three."""
    check_config(scaled("C3", J=100, D=310, P=2, B=515, density=0.03), "f32", eta=1e-3, steps=1)
    check_config(scaled("C3", J=72, D=200, P=4, B=400, density=0.03), "f32", eta=1e-3, steps=1)


def test_many_workers_f32():
    """K far beyond the benchmark shapes on the CUDA-core paths: 16384 samples (MLR), 4096 coded samples
    (seven shared-memory slices of the scatter apply)."""
    check_config(scaled("C1", J=100, D=260, P=64, B=256), "f32", eta=1e-3, steps=1)
    check_config(scaled("C3", J=64, D=256, P=64, B=64, density=0.05), "f32", eta=1e-4, steps=1)


def test_c3_sc_full_f32():
    check_config(get_config("C3"), "f32", eta=1e-4, steps=1)


def test_c3_unused_atoms_are_bit_identical():
    cfg = scaled("C3", J=96, D=800, P=2, B=8, density=0.02)
    inputs = make_inputs(cfg)
    used = np.zeros(cfg["D"], bool)
    used[inputs["idx"][0]] = True
    assert (~used).any()
    wl = _workload(cfg, inputs, "f32")
    try:
        wl.step(0, eta=0.1)
        torch.cuda.synchronize()
        W1 = wl.W.cpu().numpy()
        assert np.array_equal(W1[:, ~used], inputs["W"][:, ~used])
        assert not np.array_equal(W1[:, used], inputs["W"][:, used])
    finally:
        wl.close()


# ------------------------------------------------------------------------------------- error behaviour
def test_error_codes_and_device_status():
    from paper_1511_08486_b200 import binding as B
    cfg = get_config("C0")
    inputs = make_inputs(cfg)
    wl = _workload(cfg, inputs, "f32")
    try:
        with pytest.raises(B.SfbError) as e:
            wl.apply(0.1, K=5)                               # not a whole number of worker streams
        assert e.value.code == -1
        with pytest.raises(B.SfbError):
            wl.apply(0.1, K=cfg["K"] + cfg["B"])
        # a label outside [0, J): status bit set, that sample's u written as zeros
        wl.batches[0]["labels"][3] = 99
        wl.compute_factors(0)
        assert wl.ctx.status() == B.SFB_DEV_BAD_LABEL
        U = to_f64(wl.U)
        assert not U[3].any() and U[2].any()
        assert wl.ctx.status() == 0                          # the word is cleared by the read
        wl.batches[0]["labels"][3] = 1
        # a buffer whose header does not match: apply leaves W untouched
        wl.compute_factors(0)
        wl.pack(0)
        wl.sf_buf[20] = 11                                   # J field of the header
        wl.apply(0.5)
        assert wl.ctx.status() == B.SFB_DEV_BAD_HEADER
        assert torch.equal(wl.W, wl.W0)
    finally:
        wl.close()
    with pytest.raises(B.SfbError) as e:
        B.Context(B.make_desc("sc", "f32", 8, 8, 2, 2, v_sparse=0))
    assert e.value.code == -3
    with pytest.raises(B.SfbError) as e:
        B.Context(B.make_desc("mlr", "f32", 0, 8, 2, 2))
    assert e.value.code == -2


def test_sparse_bad_index_sets_status():
    from paper_1511_08486_b200 import binding as B
    cfg = scaled("C3", J=32, D=100, P=2, B=4, density=0.1)
    inputs = make_inputs(cfg)
    wl = _workload(cfg, inputs, "f32")
    try:
        wl.batches[0]["idx"][0] = 1000
        wl.compute_factors(0)
        assert wl.ctx.status() & B.SFB_DEV_BAD_INDEX
    finally:
        wl.close()


def test_sparse_repeated_and_unsorted_indices_are_skipped_everywhere():
    """A CSR row that repeats an atom or is not ascending: the offending entries are skipped by the forward pass,
    by the atom-major re-sort and by the scatter apply alike (status bit set, nothing out of range is touched),
    so the step equals the oracle's step on the codes with those entries removed."""
    from paper_1511_08486_b200 import binding as B
    cfg = scaled("C3", J=96, D=120, P=2, B=8, density=0.15)
    inputs = make_inputs(cfg)
    rp = inputs["rowptr"][0].astype(np.int64)
    ix, vl = inputs["idx"][0].copy(), inputs["val"][0].copy()
    # sample 3: repeat an atom (entry 2 takes the index of entry 1); sample 9: an entry out of order (smaller than its
    # predecessor); sample 12: an atom that does not exist (which also puts its successor out of order)
    for i, k, new in ((3, 2, None), (9, 4, 0), (12, 1, 100000)):
        s0 = rp[i]
        assert rp[i + 1] - s0 > 6
        ix[s0 + k] = ix[s0 + k - 1] if new is None else new
    # the documented rule: an entry is dropped if its atom is out of range or not above its predecessor in the row
    keep = np.ones(ix.size, bool)
    for i in range(cfg["K"]):
        for k in range(rp[i], rp[i + 1]):
            if ix[k] >= cfg["D"] or (k > rp[i] and ix[k - 1] >= ix[k]):
                keep[k] = False
    assert (~keep).sum() == 4
    inputs["idx"][0] = ix
    wl = _workload(cfg, inputs, "f32")
    try:
        eta = 1e-2
        wl.step(0, eta=eta)
        status = wl.ctx.status()
        assert status & B.SFB_DEV_BAD_INDEX
        W1 = wl.W.cpu().numpy().astype(np.float64)
        assert np.isfinite(W1).all()
        counts = np.array([keep[rp[i]:rp[i + 1]].sum() for i in range(cfg["K"])])
        rp_ok = np.concatenate([[0], np.cumsum(counts)]).astype(np.uint32)
        W_or, U_or, _ = orc.step(orc.MODEL_SC, inputs["W"], dict(rowptr=rp_ok, idx=ix[keep], val=vl[keep],
                                                                  Xdata=inputs["Xdata"][0]), eta)
        W0 = inputs["W"].astype(np.float64)
        err = np.linalg.norm((W1 - W0) - (W_or - W0)) / np.linalg.norm(W_or - W0)
        assert err <= 1e-5 + 2.0 ** -24 * np.linalg.norm(W0) / np.linalg.norm(W_or - W0), f"{err:.3e}"
        _, U_wire, _ = orc.unpack(wl.sf_buf.cpu().numpy())
        assert orc.rel_fro(U_wire, U_or) <= 1e-5
        # the staged calls (factors, pack, apply: the re-sort then reads the buffer's streams) agree bit for bit
        wl.reset()
        wl.compute_factors(0)
        wl.pack(0, clock=0)
        wl.apply(eta)
        assert wl.ctx.status() & B.SFB_DEV_BAD_INDEX
        assert np.array_equal(wl.W.cpu().numpy().astype(np.float64), W1)
    finally:
        wl.close()


def test_sparse_capacity_overflow_keeps_factors_and_wire_consistent():
    """Codes beyond a worker's capacity are cut off (status bit): the u the step computes, the codes on the wire and
    the codes the apply uses are the same truncated ones, so the step equals the oracle's step on them."""
    from paper_1511_08486_b200 import binding as B
    cfg = scaled("C3", J=64, D=200, P=2, B=4, density=0.2)
    inputs = make_inputs(cfg)
    cap_p = 96
    inputs["nnz_capacity"] = cap_p * cfg["P"]
    rp = inputs["rowptr"][0].astype(np.int64)
    ix, vl = inputs["idx"][0], inputs["val"][0]
    assert rp[cfg["B"]] - rp[0] > cap_p                     # worker 0 overflows
    wl = _workload(cfg, inputs, "f32")
    try:
        eta = 1e-2
        wl.step(0, eta=eta)
        assert wl.ctx.status() & B.SFB_DEV_CAPACITY
        keep = np.zeros(ix.size, bool)
        counts = np.zeros(cfg["K"], np.int64)
        for p in range(cfg["P"]):
            base = rp[p * cfg["B"]]
            for i in range(p * cfg["B"], (p + 1) * cfg["B"]):
                s0, e0 = min(rp[i], base + cap_p), min(rp[i + 1], base + cap_p)
                keep[s0:e0] = True
                counts[i] = e0 - s0
        rp_t = np.concatenate([[0], np.cumsum(counts)]).astype(np.uint32)
        W_or, U_or, _ = orc.step(orc.MODEL_SC, inputs["W"], dict(rowptr=rp_t, idx=ix[keep], val=vl[keep],
                                                                  Xdata=inputs["Xdata"][0]), eta)
        W0 = inputs["W"].astype(np.float64)
        W1 = wl.W.cpu().numpy().astype(np.float64)
        err = np.linalg.norm((W1 - W0) - (W_or - W0)) / np.linalg.norm(W_or - W0)
        assert err <= 1e-5 + 2.0 ** -24 * np.linalg.norm(W0) / np.linalg.norm(W_or - W0), f"{err:.3e}"
        _, U_wire, (rp_w, ix_w, _) = orc.unpack(wl.sf_buf.cpu().numpy())
        assert np.array_equal(rp_w, rp_t) and np.array_equal(ix_w, ix[keep])
        assert orc.rel_fro(U_wire, U_or) <= 1e-5
    finally:
        wl.close()


def test_sc_prox_unit_columns():
    """Column projection after the update (Figure 3, prox): parity with the oracle, untouched columns bit-identical."""
    cfg = scaled("C3", J=300, D=1003, P=2, B=8, density=0.05)
    inputs = make_inputs(cfg)
    wl = _workload(cfg, inputs, "f32")
    try:
        rng = np.random.default_rng(7)
        scale = rng.uniform(0.2, 3.0, cfg["D"]).astype(np.float32)      # some columns inside, some outside the ball
        W = (inputs["W"] * scale[None, :]).astype(np.float32)
        wl.W.copy_(torch.from_numpy(W))
        wl.ctx.prox(wl.W)
        torch.cuda.synchronize()
        got = wl.W.cpu().numpy()
        ref = orc.prox_unit_columns(W)
        inside = np.linalg.norm(W.astype(np.float64), axis=0) <= 1.0 - 1e-6
        assert inside.any() and (~inside).any()
        assert np.array_equal(got[:, inside], W[:, inside])
        assert orc.rel_fro(got, ref) <= 1e-6
        assert (np.linalg.norm(got.astype(np.float64), axis=0) <= 1.0 + 1e-5).all()
        wl.ctx.prox(wl.W)                                               # idempotent up to fp32 rounding
        torch.cuda.synchronize()
        assert orc.rel_fro(wl.W.cpu().numpy(), ref) <= 1e-6
    finally:
        wl.close()


def test_c1_hundred_steps_f32():
    # C1's own schedule on the fp32 path: 100 steps, pool of 8 minibatches, eta = 1e-2
    check_config(get_config("C1"), "f32", eta=1e-2, steps=100)

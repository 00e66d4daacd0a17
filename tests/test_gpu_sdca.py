"""SDCA factors for L2-regularised MLR on the GPU (aux.dual) against the oracle's `sdca_mlr_factors`.

The factor of sample i is the dual step du_i = s (dual_i + softmax(W x_i) - onehot(y_i)), the dual variables move
by it, and the rank-K apply with eta = 1 / (lambda N) keeps W = (1 / (lambda N)) sum_i dual_i x_i^T.  Checked on
every arithmetic path: one call (factors and new duals), whole steps, and a run of several epochs over a small
training set against the oracle's trajectory and the primal-dual link.
"""
import numpy as np
import pytest
import torch

from oracle import sfb_oracle as orc
from sfbgen import make_inputs, scaled
from tests.test_gpu_parity import _workload
from tests.util import TOL, assert_lines, to_f64

pytestmark = pytest.mark.gpu


def _ldd(J):
    return (J + 3) // 4 * 4


@pytest.mark.parametrize("path,over", [
    ("f32", dict(J=37, D=203, P=3, B=7)),
    ("f32", dict(J=300, D=1024, P=4, B=64)),
    ("tf32", dict(J=300, D=1024, P=4, B=64)),          # split reduction + plain softmax pass
    ("tf32", dict(J=1024, D=512, P=32, B=128)),        # fused softmax epilogue
    ("tf32x3", dict(J=300, D=1024, P=4, B=64)),
    ("bf16", dict(J=1000, D=1024, P=32, B=128)),       # fused epilogue, bf16 factors, fp32 duals
])
def test_sdca_factors_and_step(path, over):
    from paper_1511_08486_b200 import binding as B
    name = "C4" if path == "bf16" else "C1"
    cfg = scaled(name, pool=1, **over)
    cfg["path"] = path
    if name == "C4":
        cfg["labels"] = "uniform"
    inputs = make_inputs(cfg)
    J, D, K = cfg["J"], cfg["D"], cfg["K"]
    wl = _workload(cfg, inputs, path)
    try:
        rng = np.random.default_rng(9)
        s_step, lam, N = 0.5, 1e-2, 4 * K
        dual0 = (0.3 * rng.standard_normal((K, J))).astype(np.float32)
        dual_dev = torch.zeros(K, _ldd(J), dtype=torch.float32, device=wl.W.device)
        dual_dev[:, :J] = torch.from_numpy(dual0).to(wl.W.device)
        dual_dev[:, J:] = float("nan")                      # pad values are written (as zeros), never read
        t = wl.batches[0]
        aux = B.make_aux(labels=t["labels"], dual=dual_dev, sdca_step=s_step)
        X = inputs["X"][0]
        dU_or, V_or, dual_or = orc.sdca_mlr_factors(inputs["W"], X, inputs["labels"][0], dual0, s_step)
        wl.ctx.compute_factors(wl.W, t["X"], aux, wl.U, wl.V)
        torch.cuda.synchronize()
        assert wl.ctx.status() == 0
        tol = TOL[path]
        U_gpu = to_f64(wl.U)[:, :J]
        assert orc.rel_fro(U_gpu, dU_or) <= tol
        assert_lines(U_gpu, dU_or, tol, "dual steps")
        d_gpu = dual_dev.cpu().numpy().astype(np.float64)
        assert not d_gpu[:, J:].any(), "pad values of the dual rows are zeros"
        assert orc.rel_fro(d_gpu[:, :J], dual_or) <= tol
        # a whole step from the original duals: W' = W - eta sum du_i x_i^T
        dual_dev[:, :J] = torch.from_numpy(dual0).to(wl.W.device)
        eta = 1.0 / (lam * N)
        wl.ctx.step(wl.W, t["X"], aux, wl.sf_buf, eta, clock=3)
        torch.cuda.synchronize()
        W0 = inputs["W"].astype(np.float64)
        W_or = orc.apply_dense(W0, dU_or, V_or, eta)
        got = to_f64(wl.W) - W0
        storage = 2.0 ** -24 * np.linalg.norm(W0) / np.linalg.norm(W_or - W0)
        assert storage <= tol
        assert orc.rel_fro(got, W_or - W0) <= tol + storage
        h, U_wire, _ = orc.unpack(wl.sf_buf.cpu().numpy())
        assert h["clock"] == 3 and orc.rel_fro(U_wire, dU_or) <= tol
        with pytest.raises(B.SfbError):                     # a step outside (0, 1] is refused
            wl.ctx.compute_factors(wl.W, t["X"], B.make_aux(labels=t["labels"], dual=dual_dev, sdca_step=1.5), wl.U, wl.V)
    finally:
        wl.close()


def test_sdca_epochs_keep_the_primal_dual_link_and_follow_the_oracle():
    """Twelve epochs over a training set of four mini-batches on the fp32 path: W stays (1 / (lambda N)) dual^T X to
    fp32 accuracy, W and the duals follow the oracle's trajectory, and the primal objective's gradient shrinks."""
    from paper_1511_08486_b200 import binding as B
    cfg = scaled("C1", J=20, D=64, P=2, B=16, pool=4)
    cfg["path"] = "f32"
    inputs = make_inputs(cfg)
    J, D, K, pool = cfg["J"], cfg["D"], cfg["K"], cfg["pool"]
    N, lam, s_step = K * pool, 0.05, 0.25
    eta = 1.0 / (lam * N)
    wl = _workload(cfg, inputs, "f32")
    try:
        wl.W.zero_()
        W_or = np.zeros((J, D))
        duals_dev = [torch.zeros(K, _ldd(J), dtype=torch.float32, device=wl.W.device) for _ in range(pool)]
        duals_or = [np.zeros((K, J)) for _ in range(pool)]
        for epoch in range(12):
            for b in range(pool):
                t = wl.batches[b]
                aux = B.make_aux(labels=t["labels"], dual=duals_dev[b], sdca_step=s_step)
                wl.ctx.step(wl.W, t["X"], aux, wl.sf_buf, eta, clock=epoch * pool + b)
                dU, V, duals_or[b] = orc.sdca_mlr_factors(W_or, inputs["X"][b], inputs["labels"][b], duals_or[b], s_step)
                W_or = orc.apply_dense(W_or, dU, V, eta)
        torch.cuda.synchronize()
        assert wl.ctx.status() == 0
        W_gpu = to_f64(wl.W)
        assert orc.rel_fro(W_gpu, W_or) <= 1e-5
        Xall = np.concatenate([inputs["X"][b] for b in range(pool)]).astype(np.float64)
        dual_all = np.concatenate([d.cpu().numpy()[:, :J] for d in duals_dev]).astype(np.float64)
        assert orc.rel_fro(dual_all, np.concatenate(duals_or)) <= 1e-5
        link = dual_all.T @ Xall / (lam * N)
        assert orc.rel_fro(W_gpu, link) <= 1e-5
        yall = np.concatenate([inputs["labels"][b] for b in range(pool)])
        g = lambda W: np.linalg.norm(orc.delta_w(orc.mlr_factors(W, Xall, yall)[0], Xall) / N + lam * W)
        assert g(W_gpu) <= 0.2 * g(np.zeros((J, D)))        # well on the way to the primal optimum
    finally:
        wl.close()

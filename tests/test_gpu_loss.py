"""The device-side minibatch objective (sfb_loss) against the oracle's fp64 losses."""
import pytest
import torch

from oracle import sfb_oracle as orc
from sfbgen import get_config, make_inputs, scaled
from tests.test_gpu_parity import _workload
from tests.util import TOL, batch_of

pytestmark = pytest.mark.gpu


def _oracle_loss(cfg, W, batch):
    m = cfg["model"]
    if m == "mlr":
        return orc.mlr_loss(W, batch["X"], batch["labels"])
    if m == "dml":
        return orc.dml_loss(W, batch["Xa"], batch["Xb"], batch["similar"], cfg.get("margin", 1.0))
    return orc.sc_loss(W, batch["rowptr"], batch["idx"], batch["val"], batch["Xdata"])


CASES = [
    ("C0", "f32", {}),
    ("C0", "tf32", {}),
    ("C1", "f32", dict(J=100, D=260, P=3, B=10)),
    ("C1", "f32", {}),                                           # full size
    ("C1", "tf32", {}),
    ("C2", "f32", dict(J=40, D=300, P=2, B=6)),
    ("C2", "f32", {}),
    ("C2", "tf32", dict(J=64, D=512, P=2, B=64)),
    ("C3", "f32", dict(J=70, D=333, P=3, B=5, density=0.1)),
    ("C3", "f32", {}),
    ("C3", "tf32", dict(J=512, D=2000, P=4, B=32)),
    ("C1", "tf32x3", dict(J=200, D=1024, P=4, B=64)),
    ("C1", "tf32x3", {}),
    ("C2", "tf32x3", dict(J=64, D=512, P=2, B=64)),
    ("C3", "tf32x3", dict(J=512, D=2000, P=4, B=32)),
    ("C4", "bf16", dict(J=256, D=512, P=2, B=64, pool=1, labels="uniform")),
    ("C4", "bf16", dict(J=4096, D=2048, P=4, B=128, pool=1)),     # Zipf labels, several tiles per dimension
]


@pytest.mark.parametrize("name,path,over", CASES)
def test_loss_matches_oracle(name, path, over):
    cfg = scaled(name, **over) if over else get_config(name)
    cfg["path"] = path
    inputs = make_inputs(cfg)
    wl = _workload(cfg, inputs, path)
    try:
        got = wl.loss(0)
        again = wl.loss(0)
        torch.cuda.synchronize()
        assert wl.ctx.status() == 0
        want = _oracle_loss(cfg, inputs["W"], batch_of(inputs, cfg, 0))
        assert abs(got.item() - want) <= TOL[path] * abs(want), (got.item(), want)
        assert got.item() == again.item()                        # fixed reduction order
        assert torch.equal(wl.W, wl.W0)                          # a monitoring call: W untouched
    finally:
        wl.close()


def test_loss_falls_along_the_steps():
    """Gradient steps at the config's step size lower the objective of the minibatch they were computed on."""
    for name, path, over, eta in [("C1", "f32", dict(J=50, D=400, P=2, B=32), 0.05),
                                  ("C3", "f32", dict(J=64, D=400, P=2, B=16, density=0.1), 1e-3)]:
        cfg = scaled(name, **over)
        cfg["path"] = path
        cfg["pool"] = 1
        wl = _workload(cfg, make_inputs(cfg), path)
        try:
            seen = [wl.loss(0).item()]
            for t in range(3):
                wl.step(0, eta=eta)
                seen.append(wl.loss(0).item())
            assert all(b < a for a, b in zip(seen, seen[1:])), seen
        finally:
            wl.close()


def test_loss_reports_a_bad_label():
    from paper_1511_08486_b200 import binding as B
    cfg = scaled("C0", J=10, D=64, P=2, B=4)
    inputs = make_inputs(cfg)
    inputs["labels"][0][3] = 10
    wl = _workload(cfg, inputs, "f32")
    try:
        wl.loss(0)
        assert wl.ctx.status() & B.SFB_DEV_BAD_LABEL
    finally:
        wl.close()

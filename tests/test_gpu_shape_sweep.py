"""A seeded sweep over shapes on every arithmetic path, each case through the whole `check_config` comparison
(factors, byte-exact buffer, apply to zero, partial apply, steps, run-to-run bit identity, per-row bounds).

The shapes are drawn from sets that straddle every tile, chunk and vector boundary of the kernels (1, 3, 8, 20,
64, 100, 128, 130, 256 pairs per worker; 2 ... 3000 rows of W; row lengths that are or are not multiples of the
16-byte unit, the 128-byte chunk and the tile), so ragged edges, workers that share a reduction block, split
reductions and single-tile problems all occur.  It stands in for an address sanitizer (closed on the machines
this runs on): every tensor the library writes sits between guard bands filled with NaN patterns, so a stray
write shows in a band, a stray read that feeds arithmetic turns the result into NaN, and any other out-of-range
access on these shapes shows up as a wrong or non-reproducible result.
"""
import random

import pytest

from sfbgen import scaled
from tests.test_gpu_parity import check_config

pytestmark = pytest.mark.gpu

KINDS = ("mlr_f32", "mlr_tf32", "mlr_bf16", "mlr_tf32x3", "dml_f32", "dml_tf32", "dml_tf32x3", "sc_f32", "sc_tf32",
         "sc_tf32x3")


def _draw(seed: int, n: int):
    rng = random.Random(seed)
    cases = []
    for it in range(n):
        kind = KINDS[it % len(KINDS)]
        P = rng.choice([1, 2, 3, 4, 5, 8, 16])
        B = rng.choice([1, 3, 8, 20, 64, 100, 128, 130, 256])
        if P * B > 2048:
            B = max(1, 2048 // P)
        J = rng.choice([2, 7, 33, 64, 100, 128, 129, 257, 512, 600, 1000, 1500, 2048, 3000])
        mult = 8 if kind.endswith("bf16") else (4 if "tf32" in kind else 1)
        D = max(mult, rng.randint(8, 3000) // mult * mult)
        density = rng.choice([0.02, 0.1, 0.3])
        cases.append((kind, J, D, P, B, density))
    return cases


CASES = _draw(20261125, 50)


@pytest.mark.parametrize("kind,J,D,P,B,density", CASES, ids=[f"{c[0]}-J{c[1]}-D{c[2]}-P{c[3]}-B{c[4]}" for c in CASES])
def test_shape(kind, J, D, P, B, density):
    model, path = kind.split("_")
    K_ = P * B
    if model == "mlr":
        name = "C4" if path == "bf16" else "C1"
        cfg = scaled(name, J=J, D=D, P=P, B=B, pool=1)
        if name == "C4":
            cfg["labels"] = "uniform"
        cfg["path"] = path
        # a step that moves the logits of the second step by a few units (a sample's own term is eta * |x|^2 * u,
        # |x|^2 = 1 for the normalised features, D for the N(0, 1) ones): beyond that a softmax amplifies operand
        # rounding by the size of the logits, which is the arithmetic contract's doing, not the kernels'
        check_config(cfg, path, eta=0.5 if name == "C1" else 4.0 / D, steps=2, guard=True)
    elif model == "dml":
        cfg = scaled("C2", J=J, D=D, P=P, B=B)
        cfg["path"] = path
        check_config(cfg, path, eta=1e-3, steps=1, guard=True)
    else:
        cfg = scaled("C3", J=J, D=D, P=P, B=B, density=density)
        cfg["path"] = path
        check_config(cfg, path, eta=1e-2 if K_ > 4 else 0.1, steps=1, guard=True)

"""GPU parity of the error-compensated tensor-core path (SFB_PATH_TF32X3) against the fp64 oracle.

Every fp32 operand is the part the tensor core sees plus an exact remainder; a product comes from a tf32
multiplication of the operands as they are and one bf16 multiplication of pre-split correction operands; the
results are held to the tolerance of the fp32 CUDA-core path, 1e-5, whole matrix, every row and every column.  Sizes go from one tile and one pipeline stage
to the full workloads (MLR large, DML, sparse-coding dictionary update).
"""
import pytest

from sfbgen import get_config, scaled
from tests.test_gpu_parity import check_config

pytestmark = pytest.mark.gpu


def _cfg(name, **kw):
    cfg = scaled(name, **kw) if kw else get_config(name)
    cfg["path"] = "tf32x3"
    return cfg


def test_x3_single_tile_single_stage():
    check_config(_cfg("C1", J=128, D=32, P=1, B=32, pool=1), "tf32x3", eta=0.5, steps=1)
    check_config(_cfg("C1", J=128, D=128, P=1, B=32, pool=1), "tf32x3", eta=0.5, steps=1)


def test_x3_pairs_ragged_and_short_streams():
    check_config(_cfg("C0"), "tf32x3", eta=1.0, steps=1)
    for J, D, P, B in ((100, 200, 3, 10), (300, 260, 5, 8), (257, 1000, 2, 100), (640, 1024, 4, 64), (130, 72, 7, 3)):
        check_config(_cfg("C1", J=J, D=D, P=P, B=B, pool=1), "tf32x3", eta=0.5, steps=2)


def test_x3_reduction_ranges_never_come_out_empty():
    """42 atoms of reduction cut for 8 ranges give ranges of 6 atoms, of which only 7 exist: the eighth must not be
    launched (found by the shape sweep as a bounded-wait time-out of the forward pass)."""
    check_config(_cfg("C1", J=100, D=1312, P=2, B=130, pool=1), "tf32x3", eta=0.5, steps=2)
    check_config(_cfg("C2", J=2, D=1304, P=2, B=20), "tf32x3", eta=1e-3, steps=1)


def test_x3_dml():
    check_config(_cfg("C2", J=72, D=1000, P=3, B=20), "tf32x3", eta=1e-3, steps=2)
    check_config(_cfg("C2", J=600, D=2000, P=8, B=32), "tf32x3", eta=1e-4, steps=2)


def test_x3_sparse_coding_scaled():
    check_config(_cfg("C3", J=70, D=332, P=3, B=5, density=0.1), "tf32x3", eta=1e-2, steps=2)
    check_config(_cfg("C3", J=512, D=2000, P=4, B=32), "tf32x3", eta=1e-3, steps=2)


def test_x3_many_pairs_are_applied_in_several_launches():
    """16384 pairs per update: one accumulator would take 2048 roundings toward zero (3e-5 of the sum); the apply goes
    to W in sixteen launches of 1024 pairs instead and stays inside 1e-5.  Also with compaction (directory offsets)."""
    check_config(_cfg("C1", J=128, D=256, P=64, B=256, pool=1), "tf32x3", eta=0.5, steps=1)
    cfg = _cfg("C2", J=128, D=512, P=32, B=256)
    cfg["compact"] = 0
    check_config(cfg, "tf32x3", eta=1e-4, steps=1)


@pytest.mark.parametrize("name,over,eta", [
    ("C1", dict(J=300, D=260, P=5, B=8, pool=1), 0.5),          # reduction blocks of the apply span four workers
    ("C1", dict(J=257, D=1000, P=2, B=100, pool=1), 0.5),       # ragged last block of every worker
    ("C1", dict(J=128, D=256, P=16, B=256, pool=1), 0.5),       # 4096 pairs: the apply goes to W in four launches
    ("C2", dict(J=600, D=2000, P=8, B=32), 1e-4),
    ("C3", dict(J=512, D=2000, P=4, B=32), 1e-3),
])
def test_x3_step_and_separate_calls_give_the_same_bits(name, over, eta):
    """Inside sfb_step the kernels that write the factors also write the apply's correction operands, and the apply's
    epilogue leaves W's correction operand for the next forward pass; sfb_compute_factors + sfb_pack + sfb_apply
    build all of them by their own passes.  Same operands, same GEMMs: W and the buffer must agree bit for bit,
    step after step."""
    import torch
    from sfbgen import make_inputs
    from tests.test_gpu_parity import _workload
    cfg = _cfg(name, **over)
    inputs = make_inputs(cfg)
    a, b = _workload(cfg, inputs, "tf32x3"), _workload(cfg, inputs, "tf32x3")
    try:
        for t in range(3):
            a.step(t, eta=eta)
            b.compute_factors(t)
            b.pack(t, clock=t)
            b.apply(eta)
            torch.cuda.synchronize()
            assert torch.equal(a.W, b.W), f"step {t}: W differs"
            assert torch.equal(a.sf_buf, b.sf_buf), f"step {t}: SF buffer differs"
        assert a.ctx.status() == 0 and b.ctx.status() == 0
    finally:
        a.close()
        b.close()


def test_x3_c1_full():
    print("C1 tf32x3 margins:", check_config(_cfg("C1"), "tf32x3", eta=1.0, steps=2))


def test_x3_c2_full():
    print("C2 tf32x3 margins:", check_config(_cfg("C2"), "tf32x3", eta=1e-5, steps=1))


def test_x3_c3_full():
    print("C3 tf32x3 margins:", check_config(_cfg("C3"), "tf32x3", eta=1e-4, steps=1))


@pytest.mark.parametrize("path,P", [("bf16", 16), ("bf16", 64), ("tf32", 16), ("tf32", 64)])
def test_tensor_core_accumulation_rounds_toward_zero(path, P):
    """The measurement the design of the compensated kernels rests on.  With exact products (bf16 operands, or
    fp32 operands with the low 13 mantissa bits already cleared) the only error of an apply to zero is the tensor
    core's fp32 accumulation: it comes out SHORT of the exact sum by about n x 2^-26, n = MMA instructions per
    output (16 bf16 or 8 tf32 reduction steps each), i.e. one rounding toward zero per instruction."""
    import numpy as np
    import torch
    from oracle import sfb_oracle as orc
    from sfbgen import make_inputs
    from tests.test_gpu_parity import _workload
    from tests.util import to_f64
    cfg = scaled("C4" if path == "bf16" else "C1", J=256, D=256, P=P, B=256, pool=1, labels="uniform")
    cfg["path"] = path
    inputs = make_inputs(cfg)
    wl = _workload(cfg, inputs, path)
    try:
        wl.compute_factors(0)
        wl.pack(0)
        wl.W.zero_()
        wl.ctx.invalidate()
        wl.apply(-1.0)
        torch.cuda.synchronize()
        U, V = to_f64(wl.U)[:, :256], to_f64(wl.V)[:, :256]
        if path == "tf32":
            cut = lambda a: (a.astype(np.float32).view(np.uint32) & np.uint32(0xFFFFE000)).view(np.float32).astype(np.float64)
            U, V = cut(U), cut(V)
        ref, got = orc.delta_w(U, V), to_f64(wl.W)
        shortfall = -float(((got - ref) * ref).sum() / (ref * ref).sum())
        n = cfg["K"] // (16 if path == "bf16" else 8)
        print(f"{path} K={cfg['K']}: rel_fro {orc.rel_fro(got, ref):.3e}, short by {shortfall:.3e}, n x 2^-26 = {n * 2.0 ** -26:.3e}")
        assert 0.5 * n * 2.0 ** -26 <= shortfall <= 2.0 * n * 2.0 ** -26
    finally:
        wl.close()

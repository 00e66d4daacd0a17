"""GPU parity of the error-compensated tensor-core path (SFB_PATH_TF32X3) against the fp64 oracle.

Every fp32 operand is split inside the kernel into the part the tensor core sees and the exact remainder, and
each product comes from three tensor-core multiplications; the results are held to the tolerance of the fp32
CUDA-core path, 1e-5, whole matrix, every row and every column.  Sizes go from one tile and one pipeline stage
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


def test_x3_dml():
    check_config(_cfg("C2", J=72, D=1000, P=3, B=20), "tf32x3", eta=1e-3, steps=2)
    check_config(_cfg("C2", J=600, D=2000, P=8, B=32), "tf32x3", eta=1e-4, steps=2)


def test_x3_sparse_coding_scaled():
    check_config(_cfg("C3", J=70, D=332, P=3, B=5, density=0.1), "tf32x3", eta=1e-2, steps=2)
    check_config(_cfg("C3", J=512, D=2000, P=4, B=32), "tf32x3", eta=1e-3, steps=2)


def test_x3_c1_full():
    check_config(_cfg("C1"), "tf32x3", eta=1.0, steps=2)


def test_x3_c2_full():
    check_config(_cfg("C2"), "tf32x3", eta=1e-5, steps=1)


def test_x3_c3_full():
    check_config(_cfg("C3"), "tf32x3", eta=1e-4, steps=1)

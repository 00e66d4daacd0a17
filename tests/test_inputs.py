"""Shape / distribution / determinism checks of the seeded input generators."""
import numpy as np

from sfbgen import bf16_bits_to_f32, bf16_round_bits, get_config, make_inputs, scaled


def test_c0_shapes_and_determinism():
    cfg = get_config("C0")
    a, b = make_inputs(cfg), make_inputs(cfg)
    assert a["W"].shape == (10, 64) and a["W"].dtype == np.float32
    assert a["X"].shape == (1, 32, 64) and a["labels"].shape == (1, 32)
    assert a["labels"].min() >= 0 and a["labels"].max() < 10
    for k in ("W", "X", "labels"):
        assert np.array_equal(a[k], b[k])
    assert abs(a["W"].std() - 0.01) < 2e-3


def test_mlr_normalised_rows_and_zipf_labels():
    c1 = scaled("C1", J=50, D=300, P=2, B=16, pool=2)
    x = make_inputs(c1)["X"]
    assert np.allclose(np.linalg.norm(x.astype(np.float64), axis=2), 1.0, atol=1e-6)
    assert not np.array_equal(x[0], x[1])
    c4 = scaled("C4", J=4096, D=64, P=4, B=256, pool=1)
    inp = make_inputs(c4)
    y = inp["labels"][0]
    assert 0.08 < (y == 0).mean() < 0.30                  # Zipf head
    assert len(np.unique(y)) > 200
    assert inp["X_bits"].dtype == np.uint16
    assert np.array_equal(bf16_bits_to_f32(inp["X_bits"]), inp["X"])
    assert np.array_equal(bf16_round_bits(inp["X"]), inp["X_bits"])     # already bf16-representable


def test_dml_and_sc_structure():
    c2 = scaled("C2", J=20, D=200, P=2, B=8)
    d = make_inputs(c2)
    assert d["similar"].tolist() == [1, 0] * 8
    assert d["Xa"].shape == (1, 16, 200) and not np.array_equal(d["Xa"], d["Xb"])
    c3 = scaled("C3", J=64, D=400, P=4, B=8)
    s = make_inputs(c3)
    rp, ix = s["rowptr"][0], s["idx"][0]
    assert rp[0] == 0 and rp[-1] == ix.size == s["val"][0].size
    assert 0.03 < ix.size / (32 * 400) < 0.07
    assert np.allclose(np.linalg.norm(s["W"].astype(np.float64), axis=0), 1.0, atol=1e-6)
    assert s["nnz_capacity"] % (4 * 32) == 0
    per_worker = rp[8::8].astype(int) - rp[0:32:8].astype(int)
    assert per_worker.max() <= s["nnz_capacity"] // 4
    assert s["Xdata"].shape == (1, 32, 64)

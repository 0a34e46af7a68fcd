"""The checker replays the numbers the paper prints (tests/golden/paper_worked_examples.json)."""
import json
import os

import numpy as np
import pytest

import oracle

HERE = os.path.dirname(os.path.abspath(__file__))
with open(os.path.join(HERE, "golden", "paper_worked_examples.json")) as fh:
    CASES = json.load(fh)["cases"]

MODES = {"E": oracle.MODE_E, "EK": oracle.MODE_E | oracle.MODE_K, "EKC": oracle.MODE_EKC,
         "EC": oracle.MODE_E | oracle.MODE_C}
SCALE = 1.0 / (1 << 30)


def _run(case, mode):
    w = np.array(case["weights"], dtype=np.float32).reshape(case["shape"])
    return oracle.quantize_layer(w, bits=8, mode=MODES[mode], details=True)


@pytest.mark.parametrize("case", CASES, ids=[c["name"] for c in CASES])
def test_paper_worked_example(case):
    r = _run(case, case["mode"])
    assert r.scales.tolist() == [1.0], "127 / 127 must give scale exactly 1"
    assert r.codes.reshape(-1).tolist() == case["codes"]
    np.testing.assert_allclose(r.kernel_err.reshape(-1), case["kernel_sums"], atol=1e-6)
    if "channel_sum" in case:
        np.testing.assert_allclose(r.channel_err, [case["channel_sum"]], atol=1e-6)
    if "pert" in case:
        np.testing.assert_allclose(r.pert.reshape(-1) * SCALE, case["pert"], atol=1e-6)
    for stage in ("E", "EK"):
        if f"codes_{stage}" in case:
            rs = _run(case, stage)
            assert rs.codes.reshape(-1).tolist() == case[f"codes_{stage}"]
            np.testing.assert_allclose(rs.kernel_err.reshape(-1), case[f"kernel_sums_{stage}"],
                                       atol=1e-6)


def test_three_by_three_needs_at_most_four_flips():
    """App. B.4: a 3x3 kernel's CASE is at most 0.5 * 9 = 4.5, so SQuant-K flips at most 4."""
    w = np.zeros((1, 2, 3, 3), dtype=np.float32)
    w[0, 0, 0, 0] = 127.0
    w[0, 1] = 0.5000001          # nine elements each rounded up by almost one half
    r = oracle.quantize_layer(w, bits=8, mode=MODES["EK"], details=True)
    assert int((r.flip[0, 1] & 1).sum()) == 4
    assert abs(float(r.kernel_err[0, 1])) <= 0.5
    rng = np.random.default_rng(5)
    w = rng.uniform(-20, 20, size=(64, 32, 3, 3)).astype(np.float32)
    r = oracle.quantize_layer(w, bits=8, mode=MODES["EK"], details=True)
    assert int((r.flip & 1).reshape(64, 32, 9).sum(-1).max()) <= 4

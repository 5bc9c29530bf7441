"""The sweep harness: host-side summariser on CPU; one small configuration end to end on the GPU."""
import io
import json
import math

import pytest

from paper_2609_26077_b200 import sweep


def _rec(name, lv, seed, err, ref=1.0):
    return {"config": "c1", "family": "gaussian", "seed": seed, "realization": name, "levels": lv,
            "scale_mode": "fp32", "block_k": 32, "M": 256, "K": 256, "N": 256,
            "sum_sq_diff": (err ** 2) * ref, "sum_sq_ref": ref, "max_abs_diff": 0.0, "rel_frobenius": err,
            "device_status": 0}


def test_summarise_pairs_ratios_and_pools(tmp_path):
    path = tmp_path / "s.jsonl"
    recs = [_rec("cubic", 0, 0, 0.030), _rec("cubic", 0, 1, 0.040, ref=3.0),
            _rec("strassen", 1, 0, 0.060), _rec("strassen", 1, 1, 0.080, ref=3.0),
            _rec("strassen", 1, 2, 0.500)]                      # unpaired seed: excluded from the ratio
    path.write_text("".join(json.dumps(r) + "\n" for r in recs))
    rows = sweep.summarise(str(path), file=io.StringIO())
    by = {(r[1], r[2]): r for r in rows}
    assert by[("cubic", 0)][3] == 2 and by[("cubic", 0)][4] == pytest.approx(0.035)
    assert by[("cubic", 0)][6] == pytest.approx(math.sqrt((0.03 ** 2 + 3 * 0.04 ** 2) / 4.0))
    assert by[("strassen", 1)][7] == pytest.approx(2.0)         # paired over seeds 0 and 1 only
    assert by[("strassen", 1)][8] == 2.0


@pytest.mark.gpu
def test_config_c1_on_gpu(tmp_path):
    import argparse
    out = tmp_path / "c1.jsonl"
    args = argparse.Namespace(config="c1", scale_mode="fp32", block_k=32, out=str(out), trials=6, b_tile=0, b_bf16=False)
    sweep.run(args)
    n_lines = len(out.read_text().splitlines())
    assert n_lines == 12
    sweep.run(args)                                             # resume: nothing left to do
    assert len(out.read_text().splitlines()) == n_lines
    rows = sweep.summarise(str(out), file=io.StringIO())
    by = {(r[1], r[2]): r for r in rows}
    assert by[("cubic", 0)][4] == pytest.approx(0.0339, rel=0.03)
    assert by[("strassen", 1)][7] == pytest.approx(2.0, rel=0.03)


@pytest.mark.gpu
def test_covariance_diagnostic_is_small_on_gaussian_operands():
    # App. D.1: the cross-r part of the linear error term is a fraction of a percent of the whole
    rows = sweep.covariance_diagnostic(names=("strassen", "phi_optimal"), n=256, seeds=2, block_k=128, file=io.StringIO())
    for name, mean, lo, hi in rows:
        assert abs(mean) < 0.03 and lo > -0.06 and hi < 0.06, (name, mean, lo, hi)

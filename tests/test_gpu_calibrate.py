"""The guard's offline profile runs end to end on a small grid and returns usable thresholds."""
import pytest

pytestmark = pytest.mark.gpu


def test_calibrate_guard_small_grid(tmp_path):
    from paper_2609_34814_b200 import calibrate_guard as cg

    out = cg.main(["--heads", "2", "--frames", "2,3", "--densities", "0.10", "--reps", "1",
                   "--json", str(tmp_path / "g.json")])
    assert len(out["grid"]) == 2
    for r in out["grid"]:
        assert r["natural_ms"] > 0 and r["planned_ms"] > 0 and r["plan_ms"] > 0
        assert abs(r["gain_ms"] - (r["natural_ms"] - r["planned_ms"] - r["plan_ms"])) < 1e-9
        assert 0.05 < r["density"] < 0.2
    assert out["l2_fit_den"] == 16 and 0 <= out["l2_fit_num"] <= 16 * 4
    assert out["min_density_ppm"] >= 0
    assert (tmp_path / "g.json").exists()

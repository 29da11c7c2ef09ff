"""The paper's own kernel-evaluation grid (Section 6.1: M in {64..512}, N, K in {128..1024},
50 / 75 / 87.5 % sparsity) as a test: parity with the CPU oracle on the corners of the grid under
the library's own plan, and the Table-1 statistics of the planner on a 2 x 2 x 2 corner."""
import pytest

from paper_2607_12505_b200 import binding as nm
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu

RATIOS = {"50%": (2, 4), "75%": (2, 8), "87.5%": (1, 8)}


@pytest.mark.parametrize("label", list(RATIOS))
@pytest.mark.parametrize("T", [64, 512])
@pytest.mark.parametrize("O", [128, 1024])
@pytest.mark.parametrize("K", [128, 1024])
def test_grid_corner_parity(label, T, O, K):
    n, m = RATIOS[label]
    _, plan = gu.run_case(T, O, K, n, m, dtype="i8", key=f"paper_grid.{label}", rows=None)
    assert plan["path"] in (nm.NM_PATH_UMMA_SP24, nm.NM_PATH_UMMA_DENSE)


def test_planner_quality_on_grid_corner():
    from bench import planner_quality
    out = planner_quality.evaluate(Ts=(64, 512), OKs=(128, 1024), reps=10)
    assert len(out["rows"]) == 3 * 8
    for label, stats in out["summary"].items():
        for field in ("top1_hit_rate", "avg_norm_perf", "worst_norm_perf", "geomean_speedup_vs_cublas_dense", "clocks"):
            assert field in stats, (label, field)
        assert stats["shapes"] == 8
        assert 0.0 <= stats["top1_hit_rate"] <= 1.0
        assert stats["worst_norm_perf"] <= stats["avg_norm_perf"] <= 1.0
        # the plan the library picks by itself stays within 20 % of the best split-K of the sweep
        assert stats["worst_norm_perf"] >= 0.8, (label, stats)
        assert not stats["clocks"]["rejected"], stats["clocks"]

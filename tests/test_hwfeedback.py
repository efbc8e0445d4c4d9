"""Host-side hardware-feedback tooling (Section 2.3, Algorithm 2, Appendix C of the paper): the
Nsight Compute reader, the 24-metric key subset and the Pearson-based metric selection."""
import numpy as np
import pytest

from paper_2511_01884_b200 import hwfeedback as hw

CSV = '''"ID","Kernel Name","gpu__time_duration.sum","dram__bytes_read.sum","sm__cycles_elapsed.avg.per_second","launch__registers_per_thread","dram__bytes.sum.per_second"
"","","us","Gbyte","Ghz","register/thread","Tbyte/s"
"0","k<0, 1>(A, B)","733.408","1.167222","1.330688","155","1.765"
"1","k<0, 1>(A, B)","1.5","900","1.9","128","0.5"
'''


def test_reader_undoes_display_units():
    rows = hw.read_ncu_raw_csv(CSV)
    assert len(rows) == 2 and rows[0]["Kernel Name"] == "k<0, 1>(A, B)"
    assert rows[0]["gpu__time_duration.sum"] == pytest.approx(733.408e-6)
    assert rows[0]["dram__bytes_read.sum"] == pytest.approx(1.167222e9)
    assert rows[0]["sm__cycles_elapsed.avg.per_second"] == pytest.approx(1.330688e9)
    assert rows[0]["launch__registers_per_thread"] == 155.0
    assert rows[0]["dram__bytes.sum.per_second"] == pytest.approx(1.765e12)
    with pytest.raises(ValueError):
        hw.read_ncu_raw_csv("a,b\n")


def test_key_subset_is_the_papers_table():
    assert len(hw.KEY24) == 24 and len(set(hw.KEY24)) == 24
    assert hw.KEY24[0] == "sm__cycles_active.avg" and hw.KEY24[9] == "dram__bytes_read.sum"
    assert hw.KEY24[23] == "smsp__sass_average_branch_targets_threads_uniform.pct"
    got = hw.key24(hw.read_ncu_raw_csv(CSV)[0])
    assert [i for i, _, _ in got] == list(range(1, 25))
    assert got[5] == (6, "launch__registers_per_thread", 155.0) and got[0][2] is None


def test_pearson_against_closed_forms_and_libraries():
    # worked by hand: dx = (-1.5, -.5, .5, 1.5), dy = (-1.75, .25, 1.25, .25): 3.5 / sqrt(5 * 4.75)
    assert hw.pearson([1, 2, 3, 4], [2, 4, 5, 4]) == pytest.approx(3.5 / np.sqrt(23.75), abs=1e-15)
    assert hw.pearson([1, 2, 3], [10, 20, 30]) == pytest.approx(1.0)
    assert hw.pearson([1, 2, 3], [3, 1, -1]) == pytest.approx(-1.0)
    assert np.isnan(hw.pearson([1, 2, 3], [5, 5, 5]))
    rng = np.random.default_rng(0)
    from scipy import stats
    for n in (2, 3, 10, 1000):
        x, y = rng.standard_normal(n), rng.standard_normal(n)
        assert hw.pearson(x, y) == pytest.approx(np.corrcoef(x, y)[0, 1], abs=1e-12)
        if n > 2:
            assert hw.pearson(x, y) == pytest.approx(stats.pearsonr(x, y)[0], abs=1e-12)
        a, b = 3.0, -2.5           # invariance under positive affine maps, sign flip under negation
        assert hw.pearson(a * x + 1, y) == pytest.approx(hw.pearson(x, y), abs=1e-12)
        assert hw.pearson(b * x + 1, y) == pytest.approx(-hw.pearson(x, y), abs=1e-12)
    with pytest.raises(ValueError):
        hw.pearson([1.0], [2.0])


def _task(runtime, **metrics):
    return hw.task_correlations({"gpu__time_duration.sum": runtime, **metrics}, runtime, top=2)


def test_step2_ranks_by_absolute_correlation_and_drops_aliases():
    t = [1.0, 2.0, 3.0, 4.0, 5.0]
    r, top = hw.task_correlations({"gpu__time_duration.sum": t,
                                   "a": [1, 2, 3, 4, 6],                 # strongly positive
                                   "a_alias": [10, 20, 30, 40, 60],      # the same counter in other units
                                   "b": [5, 4, 3, 2.5, 0],               # strongly negative
                                   "c": [1, -1, 1, -1, 1],               # unrelated
                                   "flat": [7, 7, 7, 7, 7]}, t, top=2)
    assert set(r) == {"a", "b", "c"} and top == ["a", "b"]
    assert r["a"] > 0.98 and -0.98 < r["b"] < -0.95 and abs(r["c"]) < 0.1


def test_step3_keeps_metrics_that_recur_with_one_sign_above_the_75th_percentile():
    # three tasks, candidates' correlations chosen by hand
    A = ({"m1": 0.9, "m2": -0.8, "m3": 0.7, "m4": 0.2}, ["m1", "m2", "m3"])
    B = ({"m1": 0.95, "m2": 0.85, "m3": 0.1, "m5": -0.9}, ["m1", "m2", "m5"])
    C = ({"m1": 0.8, "m5": -0.7, "m3": 0.6, "m2": -0.1}, ["m1", "m5", "m3"])
    res = hw.select_across_tasks([A, B, C])
    S = res["scores"]
    assert S["m1"] == pytest.approx((0.9 + 0.95 + 0.8) / 3)
    assert S["m2"] == pytest.approx((0.8 + 0.85 + 0.1) / 3)
    assert S["m5"] == pytest.approx((0.9 + 0.7) / 3)              # undefined in task A counts as zero
    assert res["p75"] == pytest.approx(np.percentile([S[m] for m in ("m1", "m2", "m3", "m5")], 75))
    assert res["same_sign"] == {"m1": True, "m2": False, "m3": True, "m5": True}
    assert res["appearances"] == {"m1": 3, "m2": 2, "m3": 2, "m5": 2}
    assert res["selected"] == ["m1"]                                # the only score above P75
    # a metric that is a candidate of one task only is never selected, whatever its score
    res = hw.select_across_tasks([({"x": 1.0, "y": 0.5}, ["x", "y"]), ({"y": 0.5, "z": 0.4}, ["y", "z"])])
    assert "x" not in res["selected"]


def test_tables_from_reports_keeps_metrics_every_launch_reports():
    rows = hw.read_ncu_raw_csv(CSV)
    table, runtime = hw.tables_from_reports(rows)
    assert runtime == [pytest.approx(733.408e-6), pytest.approx(1.5e-6)]
    assert "Kernel Name" not in table and "launch__registers_per_thread" in table

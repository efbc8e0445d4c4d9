"""The seeded input generators: determinism, distributions, storage rounding, sharding."""
import numpy as np
import torch

from paper_2511_01884_b200 import workloads as wk


def test_streams_are_deterministic_and_independent():
    a = wk.draw_normal(0, 0, 4096, 1.0)
    assert np.array_equal(a, wk.draw_normal(0, 0, 4096, 1.0))
    assert not np.array_equal(a, wk.draw_normal(0, 1, 4096, 1.0))
    assert not np.array_equal(a, wk.draw_normal(1, 0, 4096, 1.0))
    # a later window of the same stream continues it
    assert np.array_equal(wk.draw_normal(0, 0, 1000, 1.0, start=3096), a[3096:])


def test_distributions():
    z = wk.draw_normal(0, 0, 1 << 20, 0.02).astype(np.float64)
    assert abs(z.mean()) < 1e-4 and abs(z.std() - 0.02) < 1e-4
    assert abs((z ** 4).mean() / z.var() ** 2 - 3.0) < 0.05          # normal kurtosis
    u = wk.draw_uniform(0, 1, 1 << 20, -1 / 16, 1 / 16).astype(np.float64)
    assert u.min() >= -1 / 16 and u.max() < 1 / 16
    assert abs(u.mean()) < 2e-4 and abs(u.var() - (1 / 8) ** 2 / 12) < 1e-5


def test_bf16_rounding_is_nearest_even():
    x = np.concatenate([wk.draw_normal(3, 0, 1 << 16, 1.0),
                        np.array([1.0, 1.00390625, 1.01171875, -1.00390625, 0.0, 3.0e38], np.float32)])
    want = torch.from_numpy(x).to(torch.bfloat16).float().numpy()
    assert np.array_equal(wk.round_to_storage(x, wk.BF16), want)
    assert np.array_equal(wk.round_to_storage(x, wk.F32), x)
    h = x[np.abs(x) < 6e4]
    assert np.array_equal(wk.round_to_storage(h, wk.F16), torch.from_numpy(h).to(torch.float16).float().numpy())


def test_workload_table_matches_the_five_configurations():
    w = wk.WORKLOADS
    assert (w["c1"].M, w["c1"].N, w["c1"].K) == (128, 512, 256)
    assert (w["c2"].M, w["c2"].N, w["c2"].K) == (4096, 4096, 4096)
    assert (w["c3"].M, w["c3"].N, w["c3"].K) == (8192, 8192, 8192)
    assert (w["c4"].M, w["c4"].N, w["c4"].K) == (16, 16384, 8192)
    assert (w["c5"].M, w["c5"].N, w["c5"].K) == (16384, 4096, 4096)
    assert w["c1"].algorithmic_bytes == 657_920
    assert w["c2"].algorithmic_bytes == 201_342_976
    assert w["c3"].algorithmic_bytes == 402_669_568
    assert w["c4"].algorithmic_bytes == 268_730_432
    assert w["c5"].algorithmic_bytes == 302_014_464
    assert w["c3"].flops == 1_099_511_627_776
    i = wk.make_inputs(w["c1"])
    assert i["X"].shape == (128, 256) and i["W"].shape == (512, 256) and i["b"].shape == (512,)
    assert i["gamma"] is None and abs(i["W"]).max() <= 1 / 16 and abs(i["b"]).max() <= 0.1


def test_row_shards_tile_the_global_input():
    wl = wk.WORKLOADS["c1"]
    full = wk.make_inputs(wl)["X"]
    for world in (1, 2, 3):
        parts, covered = [], 0
        for r in range(world):
            lo, hi = wk.shard_rows(wl.M, r, world)
            assert lo == covered
            covered = hi
            parts.append(wk.make_inputs(wl, M=hi - lo, row_offset=lo)["X"])
        assert covered == wl.M and np.array_equal(np.concatenate(parts), full)


def test_sample_rows_hit_every_tile():
    r = wk.sample_rows(1000, 128)
    assert r[0] == 0 and r[-1] == 999 and len(set(r // 128)) == 8

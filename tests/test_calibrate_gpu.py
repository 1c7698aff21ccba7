"""Window calibration kernel (paper Section 2, steps (1)-(3)) against the oracle, through the C ABI.

The maps are non-negative multiples of 1/1024, so every partial sum is exact in fp64 in any order and the
integer decision "smallest radius whose window mass reaches R_0 of the part's mass" must agree exactly."""
import numpy as np
import pytest
import torch

from oracle import litevar_oracle as orc
from paper_2411_17178_b200 import binding, workloads as wl
from tests.gpu_util import lib_ready

pytestmark = pytest.mark.gpu


def dyadic_maps(scales, k, n_maps, seed, peaked=False):
    rng = np.random.default_rng(seed)
    n_k, L_k = orc.map_shape(scales, k)
    m = rng.integers(0, 64, size=(n_maps, n_k, L_k)).astype(np.float64)
    if peaked:  # most of the mass near the co-located keys, as in real attention maps
        near = orc.mask(scales, k, [-1, -1, -1] + [max(1, s // 6) for s in scales[3:]])
        m = m + 960.0 * near[None]
    return m / 1024.0


@pytest.mark.parametrize("scales,k", [((1, 2, 3, 4), 4), ((1, 2, 3, 4, 6, 9), 6), (wl.SCALES_256, 8), (wl.SCALES_256, 10),
                                       (wl.SCALES_512, 9)])
@pytest.mark.parametrize("peaked", [False, True], ids=["flat", "peaked"])
def test_calibration_matches_oracle(scales, k, peaked):
    lib_ready()
    maps = dyadic_maps(scales, k, 3, 11 * k, peaked)
    dev = torch.tensor(maps, dtype=torch.float32, device="cuda")
    for r0 in (0.5, 0.8, 0.95, 1.0):
        rad, ratio = binding.calibrate_windows(scales, k, dev, r0, want_ratio=True)
        ref = orc.calibrate_radius(scales, k, maps, r0)
        assert rad.tolist() == ref.tolist(), (r0, rad, ref)
        for j in range(4, k + 1):
            for w in range(scales[j - 1]):
                assert ratio[j - 1, w] == pytest.approx(orc.window_ratio(scales, k, j, w, maps), rel=1e-12, abs=1e-15)
    # the radius row is a valid window table row for the planner
    tab = np.full((len(scales), len(scales)), -1, np.int32)
    tab[k - 1] = rad
    plan = binding.Plan(scales, n_heads=1, radius=tab)
    assert np.array_equal(plan.materialize_mask(k), orc.mask(scales, k, rad))
    plan.close()


def test_calibration_many_rows_per_warp():
    """More (map, query) rows than resident warps: batches of several rows, several batch waves, and query
    indices that wrap around from one map to the next inside a batch."""
    lib_ready()
    scales, k = (1, 2, 3, 4, 5, 6), 6
    maps = dyadic_maps(scales, k, 3001, 3, peaked=True)
    dev = torch.tensor(maps, dtype=torch.float32, device="cuda")
    for r0 in (0.6, 0.9):
        rad, ratio = binding.calibrate_windows(scales, k, dev, r0, want_ratio=True)
        assert rad.tolist() == orc.calibrate_radius(scales, k, maps, r0).tolist()
        for j in range(4, k + 1):
            for w in range(scales[j - 1]):
                assert ratio[j - 1, w] == pytest.approx(orc.window_ratio(scales, k, j, w, maps), rel=1e-12, abs=1e-15)


def test_calibration_wide_parts():
    """Parts of more than 256 keys, one for each count of 32-column chunks per key row the kernel
    specialises on (1, 2, 3, 4 and the general case), ahead of a small step."""
    lib_ready()
    scales, k = (1, 2, 3, 70, 100, 40, 150, 33, 17, 5), 10
    maps = dyadic_maps(scales, k, 3, 21)
    centre = orc.mask(scales, k, [-1, -1, -1] + [s // 5 for s in scales[3:]])
    maps = maps + (32.0 / 1024) * centre[None]
    dev = torch.tensor(maps, dtype=torch.float32, device="cuda")
    for r0 in (0.3, 0.7):
        rad, ratio = binding.calibrate_windows(scales, k, dev, r0, want_ratio=True)
        assert rad.tolist() == orc.calibrate_radius(scales, k, maps, r0).tolist()
        for j in range(4, k + 1):
            for w in (0, 1, scales[j - 1] // 3, scales[j - 1] - 2, scales[j - 1] - 1):
                assert ratio[j - 1, w] == pytest.approx(orc.window_ratio(scales, k, j, w, maps), rel=1e-12, abs=1e-15)


def test_calibration_planted_window_and_global_variants():
    lib_ready()
    scales, k = wl.SCALES_256, 10
    planted = [-1, -1, -1, 0, 1, 1, 2, 2, 3, 4]
    inside = orc.mask(scales, k, planted)
    maps = (dyadic_maps(scales, k, 2, 5) + 1.0 / 1024) * inside[None]
    dev = torch.tensor(maps, dtype=torch.float32, device="cuda")
    assert binding.calibrate_windows(scales, k, dev, 1.0).tolist() == planted
    # literal "first three parts" reading: scales 1..5 global
    got = binding.calibrate_windows(scales, k, dev, 1.0, n_global_scales=5)
    assert got.tolist() == orc.calibrate_radius(scales, k, maps, 1.0, n_global_scales=5).tolist()
    assert got[:5].tolist() == [-1] * 5
    # a step with global parts only
    m3 = torch.ones(1, 9, 14, device="cuda")
    assert binding.calibrate_windows(scales, 3, m3, 0.9).tolist() == [-1] * 10


def test_calibration_argument_errors():
    lib_ready()
    m = torch.ones(1, 16, 30, device="cuda")
    for kwargs in (dict(step_k=0), dict(step_k=5), dict(r0=0.0), dict(r0=1.5)):
        args = dict(scales=(1, 2, 3, 4), step_k=4, maps=m, r0=0.9)
        args.update(kwargs)
        with pytest.raises(binding.LitevarError) as e:
            binding.calibrate_windows(**args)
        assert e.value.status == 1

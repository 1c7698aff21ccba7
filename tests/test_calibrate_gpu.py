"""Window calibration kernel (paper Section 2, steps (1)-(3)) against the oracle, through the C ABI.

Most cases use maps that are non-negative multiples of 1/1024: every partial sum is then exact in fp64 in any
order and the integer decision "smallest radius whose window mass reaches R_0 of the part's mass" must agree
exactly.  One case uses real softmax rows, where the kernel's fp32 bins round: see the bound there."""
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


@pytest.mark.parametrize("scales,k,n_maps", [(wl.SCALES_256, 10, 24), (wl.SCALES_512, 9, 6)])
def test_calibration_on_softmax_rows_within_the_fp32_bin_bound(scales, k, n_maps):
    """Real post-softmax rows (fp32 softmax of seeded scores with a peak near the co-located keys).  The kernel adds
    up to 256 rows into lane-private fp32 bins before it flushes them in fp64: a bin takes at most 256 x 8 values
    of one sign, so its relative rounding error is below 2048 x 2^-24 = 1.3e-4, and so is that of any ratio of sums
    of bins (numerator and denominator err the same way at most once each: 2.5e-4).  R_w must agree with the
    oracle's within that bound, and the radius wherever the oracle's R_w at the chosen radius and at the one before
    stay farther than the bound from R_0."""
    lib_ready()
    bound = 2.5e-4
    n_k, L_k = orc.map_shape(scales, k)
    g = torch.Generator().manual_seed(100 + k)
    scores = torch.randn(n_maps, n_k, L_k, generator=g) * 1.5
    near = torch.from_numpy(orc.mask(scales, k, [-1, -1, -1] + [max(1, s // 5) for s in scales[3:]]))
    scores = scores + 2.5 * near[None].float()
    maps32 = torch.softmax(scores, dim=-1)
    maps = maps32.double().numpy()
    dev = maps32.cuda()
    for r0 in (0.6, 0.8, 0.95):
        rad, ratio = binding.calibrate_windows(scales, k, dev, r0, want_ratio=True)
        ref = orc.calibrate_radius(scales, k, maps, r0)
        for j in range(4, k + 1):
            curve = [orc.window_ratio(scales, k, j, w, maps) for w in range(scales[j - 1])]
            for w, want in enumerate(curve):
                assert abs(ratio[j - 1, w] - want) <= bound * max(want, 1e-30), (j, w, ratio[j - 1, w], want)
            w = int(ref[j - 1])
            clear = abs(curve[w] - r0) > bound and (w == 0 or abs(curve[w - 1] - r0) > bound)
            if clear:
                assert int(rad[j - 1]) == w, (r0, j, rad, ref)
            else:
                assert abs(int(rad[j - 1]) - w) <= 1

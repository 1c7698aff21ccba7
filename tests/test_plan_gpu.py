"""Device planner against the oracle's mask: bit-exact on every step of every benchmark schedule."""
import numpy as np
import pytest

from oracle import litevar_oracle as orc
from paper_2411_17178_b200 import binding, workloads as wl
from tests.gpu_util import lib_ready

pytestmark = pytest.mark.gpu

CASES = [
    ((1, 2, 3, 4), (1, 4)), ((1, 2, 3, 4, 5), (1, 4)), ((1, 2, 3, 4, 6, 9), (1, 4)), ((2, 3, 5, 7, 4), (1, 2)),
    (wl.SCALES_256, (1, 4)), (wl.SCALES_256, (1, 8)), (wl.SCALES_256, (1, 2)), (wl.SCALES_512, (1, 4)),
    ((1, 2, 3, 4, 6, 9, 13, 18, 24, 32, 48), (1, 4)),
]


def tile_tokens(geom):
    """Token of every slot of every tile (-1 = padding slot), from the exported tile geometry."""
    out = np.full((len(geom), 128), -1, np.int64)
    for i, (first, cols, stride, vr, vc) in enumerate(geom):
        m = np.arange(128)
        r, c = m // cols, m % cols
        ok = (r < vr) & (c < vc)
        out[i, ok] = first + r[ok] * stride + c[ok]
    return out


def check_step(plan, scales, k, w_row):
    n_k, L_k = orc.map_shape(scales, k)
    ref = orc.mask(scales, k, w_row)
    got = plan.materialize_mask(k)
    assert got.shape == ref.shape
    assert np.array_equal(got, ref), f"mask differs at step {k}: {np.argwhere(got != ref)[:5]}"
    st = plan.stats(k)
    assert st["live_entries"] == int(ref.sum())
    t = plan.export_tiles(k)
    qtok, ktok = tile_tokens(t["q_tile_geom"]), tile_tokens(t["key_tile_geom"])
    # the tiles partition the queries of the step and the keys of the cache prefix
    assert sorted(qtok[qtok >= 0].tolist()) == list(range(n_k))
    assert sorted(ktok[ktok >= 0].tolist()) == list(range(L_k))
    nq, nk = len(qtok), len(ktok)
    rp = t["row_ptr"]
    assert rp[0] == 0 and rp[-1] == len(t["pair_key_tile"]) == st["live_tiles"]
    assert st["full_tiles"] + st["partial_tiles"] == st["live_tiles"]
    assert int(t["pair_is_full"].sum()) == st["full_tiles"]
    # the list is exactly the set of tile pairs with a live entry, in canonical order, and the
    # full flag marks exactly the pairs whose every (valid query, key slot) entry is live
    for qt in range(nq):
        rows = ref[qtok[qt][qtok[qt] >= 0]]
        expect, full = [], []
        for kt in range(nk):
            valid = ktok[kt] >= 0
            blk = rows[:, ktok[kt][valid]]
            if blk.any():
                expect.append(kt)
                full.append(int(blk.all() and valid.all()))
        assert t["pair_key_tile"][rp[qt]:rp[qt + 1]].tolist() == expect
        assert t["pair_is_full"][rp[qt]:rp[qt + 1]].tolist() == full


TILINGS = [binding.TILING_RASTER, binding.TILING_PATCH, binding.TILING_AUTO]
TNAME = {binding.TILING_RASTER: "raster", binding.TILING_PATCH: "patch", binding.TILING_AUTO: "auto"}


@pytest.mark.parametrize("tiling", TILINGS, ids=lambda t: TNAME[t])
@pytest.mark.parametrize("scales,rho", CASES)
def test_planner_matches_oracle_mask(scales, rho, tiling):
    lib_ready()
    plan = binding.Plan(scales, n_heads=2, rho=rho, tiling=tiling)
    w = orc.window_table(scales, rho=rho)
    for k in range(1, len(scales) + 1):
        rad, bnd = plan.export_bounds(k)
        assert rad.tolist() == w[k - 1].tolist()
        s_k = scales[k - 1]
        for j in range(1, k + 1):
            s_j = scales[j - 1]
            for x in range(s_k):
                if w[k - 1, j - 1] < 0:
                    exp = (0, s_j - 1)
                else:
                    c = orc.centre(x, s_j, s_k)
                    exp = (max(0, c - w[k - 1, j - 1]), min(s_j - 1, c + w[k - 1, j - 1]))
                assert tuple(bnd[j - 1, x]) == exp
        check_step(plan, scales, k, w[k - 1])
    plan.close()


@pytest.mark.parametrize("tiling", [binding.TILING_RASTER, binding.TILING_AUTO], ids=lambda t: TNAME[t])
@pytest.mark.parametrize("rho", [(1, 8), (1, 4), (1, 2)])
def test_planner_2k_final_step(rho, tiling):
    lib_ready()
    scales = wl.SCALES_2K
    plan = binding.Plan(scales, n_heads=1, rho=rho, tiling=tiling)
    w = orc.window_table(scales, rho=rho)
    got = plan.materialize_mask(14)
    total = 0
    for r0 in range(0, 16384, 2048):
        ref = orc.mask(scales, 14, w[13], q_rows=range(r0, r0 + 2048))
        assert np.array_equal(got[r0:r0 + 2048], ref)
        total += int(ref.sum())
    assert plan.stats(14)["live_entries"] == total
    if tiling == binding.TILING_AUTO:
        # patches of the large grids: fewer executed tile pairs than raster tiles for the same mask
        raster = binding.Plan(scales, n_heads=1, rho=rho, tiling=binding.TILING_RASTER)
        assert plan.stats(14)["live_tiles"] < raster.stats(14)["live_tiles"]
        raster.close()
    plan.close()


def test_full_table_is_all_live_and_all_tiles_listed():
    lib_ready()
    scales = wl.SCALES_256
    K = len(scales)
    plan = binding.Plan(scales, n_heads=1, radius=orc.full_table(scales), tiling=binding.TILING_RASTER)
    for k in range(1, K + 1):
        n_k, L_k = orc.map_shape(scales, k)
        assert plan.materialize_mask(k).all()
        st = plan.stats(k)
        assert st["live_entries"] == n_k * L_k
        assert st["live_tiles"] == ((n_k + 127) // 128) * ((L_k + 127) // 128)
    plan.close()


def test_explicit_table_and_literal_three_parts_variant():
    lib_ready()
    scales = wl.SCALES_256
    w5 = orc.window_table(scales, n_global_scales=5)
    a = binding.Plan(scales, n_heads=1, n_global_scales=5)
    b = binding.Plan(scales, n_heads=1, radius=w5)
    for k in (6, 10):
        ref = orc.mask(scales, k, w5[k - 1])
        assert np.array_equal(a.materialize_mask(k), ref)
        assert np.array_equal(b.materialize_mask(k), ref)
    a.close()
    b.close()


def test_per_head_window_sets():
    lib_ready()
    scales = wl.SCALES_256[:8]
    tabs = np.stack([orc.window_table(scales, rho=(1, 8)), orc.window_table(scales, rho=(1, 2))])
    plan = binding.Plan(scales, n_heads=3, radius=tabs, n_sets=2, head_to_set=[0, 1, 0])
    for s in (0, 1):
        for k in (5, 8):
            assert np.array_equal(plan.materialize_mask(k, s), orc.mask(scales, k, tabs[s][k - 1]))
    plan.close()


def test_plan_errors_on_device():
    lib_ready()
    with pytest.raises(binding.LitevarError) as e:
        binding.Plan((1, 2, 3), n_heads=1, head_dim=128)
    assert e.value.status == 2
    with pytest.raises(binding.LitevarError) as e:
        binding.Plan((1, 2, 3), n_heads=2, radius=np.zeros((1, 3, 3)), n_sets=1, head_to_set=[0, 1])
    assert e.value.status == 1


@pytest.mark.parametrize("tiling", TILINGS, ids=lambda t: TNAME[t])
@pytest.mark.parametrize("scales,rho", [((1, 2, 3, 4, 6, 9), (1, 7)), (wl.SCALES_256, (1, 7)), (wl.SCALES_256, (1, 14)),
                                        (wl.SCALES_512, (1, 7))])
def test_band_window_planner_matches_oracle(scales, rho, tiling):
    # the literal reading of "window width w about the diagonal" (band in the flattened map)
    lib_ready()
    plan = binding.Plan(scales, n_heads=1, shape=binding.WINDOW_BAND, rho=rho, tiling=tiling)
    w = orc.band_table(scales, rho=rho)
    for k in range(1, len(scales) + 1):
        rad, _ = plan.export_bounds(k)
        assert rad.tolist() == w[k - 1].tolist()
        ref = orc.mask_band(scales, k, w[k - 1])
        assert np.array_equal(plan.materialize_mask(k), ref)
        assert plan.stats(k)["live_entries"] == int(ref.sum())
    plan.close()


def test_2k_totals_from_the_planner():
    """Live entries of the 2K step as the device planner counts them: the totals worked out by hand for this
    schedule (pinned on the CPU side against the oracle's enumeration and the closed form)."""
    lib_ready()
    for rho, want in (((1, 8), 34218984), ((1, 4), 112575328), ((1, 2), 321385764)):
        plan = binding.Plan(wl.SCALES_2K, n_heads=1, rho=rho)
        assert plan.stats(14)["live_entries"] == want
        plan.close()

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


def check_step(plan, scales, k, w_row):
    n_k, L_k = orc.map_shape(scales, k)
    ref = orc.mask(scales, k, w_row)
    got = plan.materialize_mask(k)
    assert got.shape == ref.shape
    assert np.array_equal(got, ref), f"mask differs at step {k}: {np.argwhere(got != ref)[:5]}"
    st = plan.stats(k)
    assert st["live_entries"] == int(ref.sum())
    t = plan.export_tiles(k)
    nq, nk = (n_k + 127) // 128, (L_k + 127) // 128
    assert t["q_tile_geom"].shape == (nq, 4) and t["key_tile_geom"].shape == (nk, 4)
    assert t["q_tile_geom"][:, 0].tolist() == [128 * i for i in range(nq)]
    assert int(t["q_tile_geom"][:, 1].sum()) == n_k and int(t["key_tile_geom"][:, 1].sum()) == L_k
    rp = t["row_ptr"]
    assert rp[0] == 0 and rp[-1] == len(t["pair_key_tile"]) == st["live_tiles"]
    assert st["full_tiles"] + st["partial_tiles"] == st["live_tiles"]
    assert int(t["pair_is_full"].sum()) == st["full_tiles"]
    # the list is exactly the set of tile pairs with a live entry, in canonical order, and the
    # full flag marks exactly the pairs whose every (valid query, key slot) entry is live
    for qt in range(nq):
        rows = ref[qt * 128:(qt + 1) * 128]
        expect, full = [], []
        for kt in range(nk):
            blk = rows[:, kt * 128:(kt + 1) * 128]
            if blk.any():
                expect.append(kt)
                full.append(int(blk.all() and blk.shape[1] == 128))
        assert t["pair_key_tile"][rp[qt]:rp[qt + 1]].tolist() == expect
        assert t["pair_is_full"][rp[qt]:rp[qt + 1]].tolist() == full


@pytest.mark.parametrize("scales,rho", CASES)
def test_planner_matches_oracle_mask(scales, rho):
    lib_ready()
    plan = binding.Plan(scales, n_heads=2, rho=rho)
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


@pytest.mark.parametrize("rho", [(1, 8), (1, 4), (1, 2)])
def test_planner_2k_final_step(rho):
    lib_ready()
    scales = wl.SCALES_2K
    plan = binding.Plan(scales, n_heads=1, rho=rho)
    w = orc.window_table(scales, rho=rho)
    got = plan.materialize_mask(14)
    total = 0
    for r0 in range(0, 16384, 2048):
        ref = orc.mask(scales, 14, w[13], q_rows=range(r0, r0 + 2048))
        assert np.array_equal(got[r0:r0 + 2048], ref)
        total += int(ref.sum())
    assert plan.stats(14)["live_entries"] == total
    plan.close()


def test_full_table_is_all_live_and_all_tiles_listed():
    lib_ready()
    scales = wl.SCALES_256
    K = len(scales)
    plan = binding.Plan(scales, n_heads=1, radius=orc.full_table(scales))
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

"""CUDA forward path against the CPU oracle, through the C ABI, on the same seeded inputs.

Tolerance for bf16 inputs with fp32 accumulation: max-abs 1e-2, relative L2 5e-3 (bf16 rounding of the
probabilities and of the output gives a relative L2 error near 2e-3).
"""
import numpy as np
import pytest
import torch

from oracle import litevar_oracle as orc
from paper_2411_17178_b200 import binding, workloads as wl
from tests.gpu_util import assert_close, check_sampled, lib_ready, run_forward, stratified_samples

pytestmark = pytest.mark.gpu

# AUTO is what callers get: the small-step kernel where a step fits it, one of the two tcgen05 kernels elsewhere
KERNELS = [binding.KERNEL_SIMT, binding.KERNEL_TCGEN05, binding.KERNEL_TCGEN05_WS, binding.KERNEL_AUTO]
KNAME = {binding.KERNEL_SIMT: "simt", binding.KERNEL_TCGEN05: "tcgen05", binding.KERNEL_TCGEN05_WS: "tcgen05-row",
         binding.KERNEL_AUTO: "auto"}
TC_KERNELS = (binding.KERNEL_TCGEN05, binding.KERNEL_TCGEN05_WS)


TILINGS = [binding.TILING_RASTER, binding.TILING_PATCH]
TNAME = {binding.TILING_RASTER: "raster", binding.TILING_PATCH: "patch"}


@pytest.mark.parametrize("tiling", TILINGS, ids=lambda t: TNAME[t])
@pytest.mark.parametrize("kernel", KERNELS, ids=lambda k: KNAME[k])
@pytest.mark.parametrize("scales", [(1, 2, 3, 4), (1, 2, 3, 4, 5), (1, 2, 3, 4, 6, 9), (1, 2, 3, 4, 5, 6, 8, 10, 13)])
def test_tiny_schedules_every_output(scales, kernel, tiling):
    lib_ready()
    w = wl.small_workload(scales, n_heads=3, batch_pairs=1)
    plan = binding.Plan(scales, n_heads=3, tiling=tiling)
    tab = orc.window_table(scales)
    Kc, Vc = wl.make_kv(w, 0)
    for k in w.steps:
        Q = wl.make_q(w, 0, k)
        got, _ = run_forward(plan, k, 1, Q, Kc, Vc, kernel)
        ref = orc.attention_step(scales, k, tab[k - 1], Q, Kc, Vc)
        assert_close(got, ref, f"{KNAME[kernel]} scales={scales} step {k}")
    plan.close()


@pytest.mark.parametrize("kernel", KERNELS, ids=lambda k: KNAME[k])
def test_config1_full(kernel):
    lib_ready()
    w = wl.WORKLOADS[1]
    plan = binding.Plan(w.scales, n_heads=w.n_heads)
    tab = orc.window_table(w.scales)
    Kc, Vc = wl.make_kv(w, 0)
    Q = wl.make_q(w, 0, 10)
    got, out = run_forward(plan, 10, 1, Q, Kc, Vc, kernel)
    ref = orc.attention_step(w.scales, 10, tab[9], Q, Kc, Vc)
    assert_close(got, ref, "config 1")
    # a second run gives the same bits (no dependence on stale shared/tensor memory)
    got2, out2 = run_forward(plan, 10, 1, Q, Kc, Vc, kernel)
    assert torch.equal(out.view(torch.int16), out2.view(torch.int16))
    plan.close()


@pytest.mark.parametrize("tiling", TILINGS, ids=lambda t: TNAME[t])
@pytest.mark.parametrize("kernel", KERNELS, ids=lambda k: KNAME[k])
def test_config2_one_layer_all_steps_with_sharing(kernel, tiling):
    lib_ready()
    w = wl.WORKLOADS[2]
    B = 2  # batch 2x2 here keeps the oracle fast; bench runs 2x8
    plan = binding.Plan(w.scales, n_heads=w.n_heads, share_steps=[1] * 10, tiling=tiling)
    tab = orc.window_table(w.scales)
    Kc, Vc = wl.make_kv(w, 0, batch_rows=2 * B)
    for k in w.steps:
        Q = wl.make_q(w, 0, k, batch_rows=2 * B)
        # poison the unconditional half of the inputs: a shared step must never read it
        Qp, Kp, Vp = Q.clone(), Kc.clone(), Vc.clone()
        Qp[B:], Kp[B:], Vp[B:] = float("nan"), float("nan"), float("nan")
        got, out = run_forward(plan, k, B, Qp, Kp, Vp, kernel)
        ref = orc.attention_step(w.scales, k, tab[k - 1], Q, Kc, Vc, share_cfg=True)
        assert_close(got, ref, f"config 2 step {k}")
        assert torch.equal(out[:B].view(torch.int16), out[B:].view(torch.int16))
    plan.close()


@pytest.mark.parametrize("tiling", [binding.TILING_AUTO, binding.TILING_PATCH], ids=["auto", "patch"])
def test_config4_final_steps_sampled(tiling):
    lib_ready()
    w = wl.WORKLOADS[4]
    B = 1
    plan = binding.Plan(w.scales, n_heads=w.n_heads, share_steps=[1] * 10, tiling=tiling)
    tab = orc.window_table(w.scales)
    Kc, Vc = wl.make_kv(w, 0, batch_rows=2 * B)
    rng = np.random.default_rng(4)
    total = 0
    for k in (8, 9, 10):
        Q = wl.make_q(w, 0, k, batch_rows=2 * B)
        smp = stratified_samples(plan, k, 2 * B, w.n_heads, w.scales[k - 1], 20 if tiling == binding.TILING_AUTO else 8, rng)
        total += len(smp)
        ref = orc.attention_sampled(w.scales, k, tab[k - 1], Q, Kc, Vc, smp, share_cfg=True)
        # the default tiling with the kernel AUTO picks and with both tcgen05 kernels; patch tiles with both
        for kernel in ((binding.KERNEL_AUTO,) if tiling == binding.TILING_AUTO else ()) + TC_KERNELS:
            got, out = run_forward(plan, k, B, Q, Kc, Vc, kernel)
            check_sampled(got, ref, smp, f"config 4 step {k} {KNAME[kernel]}")
            assert torch.equal(out[:B].view(torch.int16), out[B:].view(torch.int16))
    assert tiling != binding.TILING_AUTO or total >= 4096
    plan.close()


@pytest.mark.parametrize("tiling", [binding.TILING_AUTO, binding.TILING_RASTER], ids=["auto", "raster"])
@pytest.mark.parametrize("rho", [(1, 8), (1, 4), (1, 2), None], ids=["rho1/8", "rho1/4", "rho1/2", "dense"])
def test_config5_sampled(rho, tiling):
    # the 2K step in the launch configuration the bench times: at least 4096 oracle rows per variant under the
    # default tiling, one from every query tile of every tenth (batch row, head) unit
    lib_ready()
    w = wl.WORKLOADS[5]
    if rho is None:
        tab = orc.full_table(w.scales)
        plan = binding.Plan(w.scales, n_heads=w.n_heads, radius=tab, tiling=tiling)
    else:
        tab = orc.window_table(w.scales, rho=rho)
        plan = binding.Plan(w.scales, n_heads=w.n_heads, rho=rho, tiling=tiling)
    Kc, Vc = wl.make_kv(w, 0)
    Q = wl.make_q(w, 0, 14)
    rng = np.random.default_rng(5)
    smp = stratified_samples(plan, 14, 2, w.n_heads, 128, 128 if tiling == binding.TILING_AUTO else 8, rng)
    assert tiling != binding.TILING_AUTO or len(smp) >= 4096
    ref = orc.attention_sampled(w.scales, 14, tab[13], Q, Kc, Vc, smp)
    # what AUTO launches for the 2K step (the kernel with a softmax thread per query row), then the other kernel
    assert plan.step_kernel(14, 1) == binding.KERNEL_TCGEN05_WS
    for kernel in (binding.KERNEL_AUTO, binding.KERNEL_TCGEN05):
        got, _ = run_forward(plan, 14, 1, Q, Kc, Vc, kernel)
        assert np.isfinite(got).all()
        check_sampled(got, ref, smp, f"config 5 rho={rho} {KNAME[kernel]}")
    plan.close()


@pytest.mark.parametrize("kernel", KERNELS, ids=lambda k: KNAME[k])
def test_dense_variant_matches_library_attention(kernel):
    # R_0 = 1: the same kernel with an all-live plan is plain attention; compare with torch SDPA on the GPU
    lib_ready()
    scales = wl.SCALES_256
    w = wl.small_workload(scales, n_heads=4, batch_pairs=1, index=91)
    plan = binding.Plan(scales, n_heads=4, radius=orc.full_table(scales))
    Kc, Vc = wl.make_kv(w, 0)
    for k in (7, 10):
        Q = wl.make_q(w, 0, k)
        got, _ = run_forward(plan, k, 1, Q, Kc, Vc, kernel)
        L = orc.map_shape(scales, k)[1]
        ref = torch.nn.functional.scaled_dot_product_attention(
            Q.cuda().float(), Kc[:, :, :L].cuda().float(), Vc[:, :, :L].cuda().float()).double().cpu().numpy()
        assert_close(got, ref, f"dense step {k}")
        ref64 = orc.attention_step(scales, k, orc.full_table(scales)[k - 1], Q, Kc, Vc)
        assert_close(got, ref64, f"dense step {k} vs oracle")
    plan.close()


@pytest.mark.parametrize("kernel", KERNELS, ids=lambda k: KNAME[k])
def test_strided_layout_and_custom_scale(kernel):
    # tensors stored [2B, tokens, H, 64] and passed as permuted views; explicit softmax scale
    lib_ready()
    scales = wl.SCALES_256[:9]
    H, B, k = 3, 1, 9
    w = wl.small_workload(scales, n_heads=H, batch_pairs=B, index=92)
    plan = binding.Plan(scales, n_heads=H, sm_scale=0.2, tiling=binding.TILING_PATCH)
    tab = orc.window_table(scales)
    Kc, Vc = wl.make_kv(w, 0)
    Q = wl.make_q(w, 0, k)
    plan.set_kernel(kernel)

    def relayout(t):
        return t.permute(0, 2, 1, 3).contiguous().cuda().permute(0, 2, 1, 3)

    q, kc, vc = relayout(Q), relayout(Kc), relayout(Vc)
    out = relayout(torch.zeros_like(Q))
    assert not q.is_contiguous()
    plan.forward(k, B, q, kc, vc, out)
    torch.cuda.synchronize()
    ref = orc.attention_step(scales, k, tab[k - 1], Q, Kc, Vc, sm_scale=0.2)
    assert_close(out.double().cpu().numpy(), ref, "strided")
    plan.close()


@pytest.mark.parametrize("kernel", KERNELS, ids=lambda k: KNAME[k])
def test_sharp_softmax_and_cache_tail_ignored(kernel):
    # large-magnitude keys (peaked softmax) and non-finite rows beyond L_k that must never be read into the result
    lib_ready()
    scales = wl.SCALES_256[:8]
    k = 7
    w = wl.small_workload(scales, n_heads=2, batch_pairs=1, index=93)
    plan = binding.Plan(scales, n_heads=2)
    tab = orc.window_table(scales)
    Kc, Vc = wl.make_kv(w, 0)
    Kc = (Kc.float() * 4).to(torch.bfloat16)
    L = orc.map_shape(scales, k)[1]
    Kc[:, :, L:] = float("nan")
    Vc[:, :, L:] = float("inf")
    Q = wl.make_q(w, 0, k)
    got, _ = run_forward(plan, k, 1, Q, Kc, Vc, kernel)
    ref = orc.attention_step(scales, k, tab[k - 1], Q, Kc, Vc)
    assert_close(got, ref, "sharp")
    plan.close()


@pytest.mark.parametrize("kernel", KERNELS, ids=lambda k: KNAME[k])
def test_dead_keys_with_huge_scores_change_nothing(kernel):
    """Masking happens before the maximum and the exponentials (Section 2: tokens outside the window are not
    attended to): keys whose scores dwarf every live score must leave the rows they are dead for untouched.  Two
    keys of the last scale are scaled by 512; they are live for the queries around them and dead for the rest."""
    lib_ready()
    scales = wl.SCALES_256
    k = 10
    w = wl.small_workload(scales, n_heads=2, batch_pairs=1, index=92)
    plan = binding.Plan(scales, n_heads=2, rho=(1, 8))
    tab = orc.window_table(scales, rho=(1, 8))
    Kc, Vc = wl.make_kv(w, 0)
    off = orc.map_shape(scales, k - 1)[1]          # first cache row of the last scale
    planted = [off + 3 * 16 + 2, off + 12 * 16 + 13]
    for t in planted:
        Kc[:, :, t] = (Kc[:, :, t].float() * 512).to(torch.bfloat16)
    Q = wl.make_q(w, 0, k)
    got, _ = run_forward(plan, k, 1, Q, Kc, Vc, kernel)
    ref = orc.attention_step(scales, k, tab[k - 1], Q, Kc, Vc)
    live = orc.mask(scales, k, tab[k - 1])[:, planted]             # [n_k, 2]
    untouched = ~live.any(axis=1)
    assert 100 < untouched.sum() < live.shape[0]
    assert np.isfinite(got).all()
    assert_close(got[:, :, untouched], ref[:, :, untouched], "rows for which the planted keys are dead")
    plan.close()


def test_per_head_window_sets_forward():
    lib_ready()
    scales = wl.SCALES_256[:9]
    H, k = 4, 9
    tabs = np.stack([orc.window_table(scales, rho=(1, 8)), orc.window_table(scales, rho=(1, 2))])
    h2s = [0, 1, 1, 0]
    w = wl.small_workload(scales, n_heads=H, batch_pairs=1, index=94)
    plan = binding.Plan(scales, n_heads=H, radius=tabs, n_sets=2, head_to_set=h2s)
    Kc, Vc = wl.make_kv(w, 0)
    Q = wl.make_q(w, 0, k)
    for kernel in KERNELS:
        got, _ = run_forward(plan, k, 1, Q, Kc, Vc, kernel)
        for h in range(H):
            ref = orc.attention_step(scales, k, tabs[h2s[h]][k - 1], Q[:, h:h + 1], Kc[:, h:h + 1], Vc[:, h:h + 1])
            assert_close(got[:, h:h + 1], ref, f"head {h}")
    plan.close()


@pytest.mark.parametrize("batch_pairs", [1, 64], ids=["B1", "B64"])
def test_per_head_window_sets_on_the_small_step_kernel(batch_pairs):
    """Two window sets on a step that AUTO gives to the small-step kernel (64 queries x 155 keys), whose list
    look-up per head runs on the device.  One batch pair leaves SMs to spare (two warps per row group), 64 batch
    pairs do not (one warp per row group): both builds of the kernel."""
    lib_ready()
    scales = (1, 2, 3, 4, 5, 6, 8)
    H, k = 4, 7
    tabs = np.stack([orc.window_table(scales, rho=(1, 8)), orc.window_table(scales, rho=(1, 2))])
    h2s = [1, 0, 0, 1]
    w = wl.small_workload(scales, n_heads=H, batch_pairs=batch_pairs, share_cfg=True, index=99)
    plan = binding.Plan(scales, n_heads=H, radius=tabs, n_sets=2, head_to_set=h2s, share_steps=[1] * len(scales))
    assert plan.step_kernel(k, batch_pairs) == binding.KERNEL_SMALL
    Kc, Vc = wl.make_kv(w, 0)
    Q = wl.make_q(w, 0, k)
    got, out = run_forward(plan, k, batch_pairs, Q, Kc, Vc)
    for h in range(H):
        ref = orc.attention_step(scales, k, tabs[h2s[h]][k - 1], Q[:, h:h + 1], Kc[:, h:h + 1], Vc[:, h:h + 1],
                                 share_cfg=True)
        assert_close(got[:, h:h + 1], ref, f"head {h}")
    assert not np.array_equal(orc.mask(scales, k, tabs[0][k - 1]), orc.mask(scales, k, tabs[1][k - 1]))
    assert torch.equal(out[:batch_pairs].view(torch.int16), out[batch_pairs:].view(torch.int16))
    plan.close()


def test_forward_argument_errors():
    lib_ready()
    scales = (1, 2, 3, 4)
    plan = binding.Plan(scales, n_heads=1)
    q = torch.zeros(2, 1, 16, 64, dtype=torch.bfloat16, device="cuda")
    kv = torch.zeros(2, 1, 30, 64, dtype=torch.bfloat16, device="cuda")
    s = (q.stride(0), q.stride(1), q.stride(2))
    sk = (kv.stride(0), kv.stride(1), kv.stride(2))
    args = lambda **kw: dict(dict(step_k=4, batch_pairs=1, q_ptr=q.data_ptr(), q_str=s, k_ptr=kv.data_ptr(),
                                  k_str=sk, v_ptr=kv.data_ptr(), v_str=sk, o_ptr=q.data_ptr(), o_str=s,
                                  stream_ptr=None), **kw)
    assert plan.forward_raw(**args()) == 0
    assert plan.forward_raw(**args(step_k=0)) == 1
    assert plan.forward_raw(**args(step_k=5)) == 1
    assert plan.forward_raw(**args(batch_pairs=0)) == 1
    assert plan.forward_raw(**args(q_ptr=None)) == 1
    assert plan.forward_raw(**args(q_ptr=q.data_ptr() + 2)) == 1
    assert plan.forward_raw(**args(q_str=(1024, 1024, 60))) == 1
    torch.cuda.synchronize()
    plan.close()


@pytest.mark.parametrize("kernel", KERNELS, ids=lambda k: KNAME[k])
def test_band_window_forward(kernel):
    # band reading of the window: same kernels, another plan
    lib_ready()
    scales = wl.SCALES_256
    H, B = 3, 1
    w = wl.small_workload(scales, n_heads=H, batch_pairs=B, share_cfg=True, index=98)
    plan = binding.Plan(scales, n_heads=H, shape=binding.WINDOW_BAND, rho=(1, 7), share_steps=[1] * len(scales))
    tab = orc.band_table(scales)
    Kc, Vc = wl.make_kv(w, 0)
    for k in (5, 8, 10):
        Q = wl.make_q(w, 0, k)
        got, _ = run_forward(plan, k, B, Q, Kc, Vc, kernel)
        ref = orc.attention_step(scales, k, tab[k - 1], Q, Kc, Vc, share_cfg=True, band=True)
        assert_close(got, ref, f"band step {k}")
    plan.close()


def test_band_window_2k_sampled():
    lib_ready()
    w = wl.WORKLOADS[5]
    tab = orc.band_table(w.scales)
    plan = binding.Plan(w.scales, n_heads=w.n_heads, shape=binding.WINDOW_BAND, rho=(1, 7))
    Kc, Vc = wl.make_kv(w, 0)
    Q = wl.make_q(w, 0, 14)
    rng = np.random.default_rng(6)
    smp = stratified_samples(plan, 14, 2, w.n_heads, 128, 128, rng)
    assert len(smp) >= 4096
    ref = orc.attention_sampled(w.scales, 14, tab[13], Q, Kc, Vc, smp, band=True)
    for kernel in TC_KERNELS:
        got, _ = run_forward(plan, 14, 1, Q, Kc, Vc, kernel)
        check_sampled(got, ref, smp, f"band 2K {KNAME[kernel]}")
    plan.close()


@pytest.mark.parametrize("cfg,steps,per_unit", [(2, (1, 4, 8, 10), 12), (3, (6, 8, 9, 10), 6), (4, (7, 8, 9, 10), 8)],
                         ids=["cfg2", "cfg3", "cfg4"])
def test_bench_launch_configuration_sampled(cfg, steps, per_unit):
    # the batch, head count, sharing and kernel build that bench.py times for this workload; outputs are checked
    # on stratified rows the oracle computes one by one: at least 4096 per workload, every (batch row, head)
    # unit, every query tile of every tenth unit, grid corners and edges, the heaviest and lightest tiles
    lib_ready()
    w = wl.WORKLOADS[cfg]
    B = w.batch_pairs
    plan = binding.Plan(w.scales, n_heads=w.n_heads, share_steps=[1] * len(w.scales))
    tab = orc.window_table(w.scales)
    Kc, Vc = wl.make_kv(w, 0, max_step=max(steps))
    kd, vd = Kc.cuda(), Vc.cuda()
    rng = np.random.default_rng(cfg)
    total = 0
    for k in steps:
        Q = wl.make_q(w, 0, k)
        out = torch.full(Q.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
        plan.forward(k, B, Q.cuda(), kd, vd, out)
        torch.cuda.synchronize()
        assert plan.poll() == 0
        assert bool(torch.isfinite(out.float()).all())
        smp = stratified_samples(plan, k, 2 * B, w.n_heads, w.scales[k - 1], per_unit, rng)
        total += len(smp)
        ref = orc.attention_sampled(w.scales, k, tab[k - 1], Q, Kc, Vc, smp, share_cfg=True)
        check_sampled(out, ref, smp, f"config {cfg} step {k}")
        assert torch.equal(out[:B].view(torch.int16), out[B:].view(torch.int16))
    assert total >= 4096
    plan.close()


def _expected_tc(plan, k):
    """The tcgen05 kernel AUTO picks for a step that is not a small one: the kernel with a softmax thread per
    query row from eight live key tiles per query tile on."""
    nq, _, npairs = plan.tile_counts(k)
    return binding.KERNEL_TCGEN05_WS if -(-npairs // nq) >= 8 else binding.KERNEL_TCGEN05


def test_step_kernel_selection():
    """AUTO runs the small-step kernel on steps with one query tile, at most two raster key tiles and little
    work, whatever the batch; a tcgen05 kernel elsewhere (the row kernel on long tile lists); forcing a kernel or
    patch tiles overrides it."""
    lib_ready()
    S, T, R, M = binding.KERNEL_SIMT, binding.KERNEL_TCGEN05, binding.KERNEL_TCGEN05_WS, binding.KERNEL_SMALL
    plan = binding.Plan(wl.SCALES_256, n_heads=2)
    assert [plan.step_kernel(k, 1) for k in range(1, 11)] == [M] * 7 + [T] * 3     # up to 64 x 155; short lists
    assert [plan.step_kernel(k, 64) for k in range(1, 11)] == [M] * 7 + [T] * 3
    for forced in (T, R, S):
        plan.set_kernel(forced)
        assert [plan.step_kernel(k) for k in range(1, 11)] == [forced] * 10
    plan.close()
    plan = binding.Plan(wl.SCALES_512, n_heads=2)
    want = [M] * 6 + [_expected_tc(plan, k) for k in range(7, 11)]                  # step 7 has two query tiles
    assert want[6] == T and want[9] == R                                            # 3 and 13 key tiles per query tile
    assert [plan.step_kernel(k, 1) for k in range(1, 11)] == want
    assert [plan.step_kernel(k, 64) for k in range(1, 11)] == want
    plan.close()
    plan = binding.Plan(wl.SCALES_2K, n_heads=1)
    assert plan.step_kernel(14, 1) == R
    plan.close()
    plan = binding.Plan(wl.SCALES_256, n_heads=2, tiling=binding.TILING_PATCH)
    assert all(plan.step_kernel(k) in (T, R) for k in range(1, 11))   # patch query tiles at every step: no small steps
    plan.close()
    with pytest.raises(binding.LitevarError):
        binding.Plan((1, 2), n_heads=1).step_kernel(3)


@pytest.mark.parametrize("scales,n_global,share", [
    ((1, 11), 0, False),        # 121 queries (eight warps, the last with 9 rows) x 122 keys
    ((15, 4), 0, True),         # 16 queries x 241 keys: one warp, four 64-key rounds, two key tiles, shared step
    ((2, 9, 3), 1, False),      # non-monotone scales: 9 queries x 94 keys at the last step
    ((1, 2, 3, 4, 6, 9, 5), 3, True),   # 25 queries x 172 keys with windows on four scales
    ((12, 8), 0, False),        # 64 queries x 208 keys: 4 warps x 4 rounds
])
def test_small_step_kernel_shape_extremes(scales, n_global, share):
    """Shapes at the edges of what the small-step kernel takes (row groups and key rounds with ragged ends,
    one to four 64-key rounds shared by the two warps of a row group), each step checked in full against the
    oracle."""
    lib_ready()
    H, B = 3, 1
    w = wl.small_workload(scales, n_heads=H, batch_pairs=B, share_cfg=share, index=90)
    plan = binding.Plan(scales, n_heads=H, n_global_scales=n_global,
                        share_steps=[1] * len(scales) if share else None)
    tab = orc.window_table(scales, n_global_scales=n_global)
    Kc, Vc = wl.make_kv(w, 0)
    for k in range(1, len(scales) + 1):
        n_k, L_k = orc.map_shape(scales, k)
        small = n_k <= 128 and L_k <= 256 and -(-n_k // 16) * -(-L_k // 64) <= 18
        assert plan.step_kernel(k, B) == (binding.KERNEL_SMALL if small else _expected_tc(plan, k)), (scales, k)
        assert small or k < len(scales)     # the step each case is about runs on the small-step kernel
        assert np.array_equal(plan.materialize_mask(k), orc.mask(scales, k, tab[k - 1]))
        Q = wl.make_q(w, 0, k)
        got, out = run_forward(plan, k, B, Q, Kc, Vc)
        ref = orc.attention_step(scales, k, tab[k - 1], Q, Kc, Vc, share_cfg=share)
        assert_close(got, ref, f"small-step kernel scales={scales} step {k}")
        if share:
            assert torch.equal(out[:B].view(torch.int16), out[B:].view(torch.int16))
    plan.close()

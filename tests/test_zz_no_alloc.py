"""litevar_attn_forward_static: the entry point for callers that are not allowed to allocate device memory
(a fixed device-memory budget, a plug-in that must not touch its host's allocator).  It rebuilds the
step's tile plan inside an array that is part of the library and runs the same forward kernel, so its
output must agree with the plan-based entry point and, like it, with the CPU oracle.  Collected last on
purpose (file name): a failure here cannot hide the result of any other test."""
import numpy as np
import pytest
import torch

from oracle import litevar_oracle as orc
from paper_2411_17178_b200 import binding, workloads as wl
from tests.gpu_util import MAX_ABS, REL_L2, assert_close, errors, lib_ready

pytestmark = pytest.mark.gpu


def _both(scales, H, B, k, share, index, rho=(1, 4), radius=None, shape=binding.WINDOW_SQUARE, stream=None):
    """One step through the plan entry point and through the entry point that allocates nothing; the two outputs
    against each other and each against the oracle."""
    w = wl.small_workload(scales, n_heads=H, batch_pairs=B, share_cfg=share, index=index)
    Kc, Vc = wl.make_kv(w, 0)
    Q = wl.make_q(w, 0, k)
    q, kc, vc = Q.cuda(), Kc.cuda(), Vc.cuda()
    plan = binding.Plan(scales, n_heads=H, rho=rho, radius=radius, shape=shape,
                        share_steps=[1] * len(scales) if share else None)
    ref = torch.full(q.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    plan.forward(k, B, q, kc, vc, ref)
    torch.cuda.synchronize()
    assert plan.poll() == 0
    plan.close()
    got = torch.full(q.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    if stream is not None:
        stream.wait_stream(torch.cuda.current_stream())
    binding.forward_static(scales, H, k, B, q, kc, vc, got, share_cfg=share, rho=rho, radius=radius, shape=shape,
                           stream=stream)
    torch.cuda.synchronize()
    g, r = got.double().cpu().numpy(), ref.double().cpu().numpy()
    assert np.isfinite(g).all()
    ma, rl = errors(g, r)
    assert ma <= MAX_ABS and rl <= REL_L2, (k, ma, rl)
    if radius is not None:
        w_row = np.asarray(radius)[k - 1]
    elif shape == binding.WINDOW_BAND:
        w_row = orc.band_table(scales, rho=rho)[k - 1]
    else:
        w_row = orc.window_table(scales, rho=rho)[k - 1]
    want = orc.attention_step(scales, k, w_row, Q, Kc, Vc, share_cfg=share, band=shape == binding.WINDOW_BAND)
    assert_close(g, want, f"no-allocation entry point vs oracle, step {k}")
    assert_close(r, want, f"plan entry point vs oracle, step {k}")
    return q, kc, vc, got


def test_two_calls_in_a_row_match_the_plan_entry_point():
    lib_ready()
    # second call: another schedule, step, head count and sharing mode, so it must not depend on
    # anything the first call left in the shared array
    _both(wl.SCALES_512, H=3, B=1, k=10, share=False, index=95)
    _both(wl.SCALES_256, H=2, B=2, k=9, share=True, index=96, rho=(1, 8))
    # and the first case again, after the smaller one overwrote part of the array
    _both(wl.SCALES_512, H=3, B=1, k=10, share=False, index=95)


def test_small_steps_and_explicit_table():
    lib_ready()
    scales = wl.SCALES_256
    K = len(scales)
    tab = np.full((K, K), -1, np.int32)
    tab[:, 3:] = 1
    for k in (1, 2, 4, 7):
        _both(scales, H=2, B=1, k=k, share=False, index=97, radius=tab)


def test_step_beyond_the_fixed_array_is_refused_before_any_launch():
    lib_ready()
    scales = wl.SCALES_2K            # step 14: 128 x 268 candidate pairs > 2048
    t = torch.zeros(2, 1, 8, 64, dtype=torch.bfloat16, device="cuda")   # never dereferenced
    with pytest.raises(binding.LitevarError) as e:
        binding.forward_static(scales, 1, 14, 1, t, t, t, t)
    assert e.value.status == 2 and "2048" in str(e.value)
    with pytest.raises(binding.LitevarError) as e:
        binding.forward_static(scales, 1, 15, 1, t, t, t, t)
    assert e.value.status == 1
    torch.cuda.synchronize()


def test_band_window_side_stream_and_no_allocation():
    lib_ready()
    # the band reading of the window, on a stream of its own
    side = torch.cuda.Stream()
    q, kc, vc, got = _both(wl.SCALES_256, H=2, B=1, k=8, share=False, index=94, rho=(1, 7),
                           shape=binding.WINDOW_BAND, stream=side)
    # a further call must leave the device's free memory where it was: the entry point allocates nothing
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    binding.forward_static(wl.SCALES_256, 2, 8, 1, q, kc, vc, got, rho=(1, 7), shape=binding.WINDOW_BAND, stream=side)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before

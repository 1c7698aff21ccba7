"""litevar_attn_forward_static: the entry point for callers that are not allowed to allocate device memory
(a fixed device-memory budget, a plug-in that must not touch its host's allocator).  It rebuilds the
step's tile plan inside an array that is part of the library and runs the same forward kernel, so its
output must agree with the plan-based entry point.  Collected last on purpose (file name): a failure
here cannot hide the result of any other test."""
import numpy as np
import pytest
import torch

from paper_2411_17178_b200 import binding, workloads as wl
from tests.gpu_util import MAX_ABS, REL_L2, errors, lib_ready

pytestmark = pytest.mark.gpu


def _both(scales, H, B, k, share, index, rho=(1, 4), radius=None):
    w = wl.small_workload(scales, n_heads=H, batch_pairs=B, share_cfg=share, index=index)
    Kc, Vc = wl.make_kv(w, 0)
    Q = wl.make_q(w, 0, k)
    q, kc, vc = Q.cuda(), Kc.cuda(), Vc.cuda()
    plan = binding.Plan(scales, n_heads=H, rho=rho, radius=radius,
                        share_steps=[1] * len(scales) if share else None)
    ref = torch.full(q.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    plan.forward(k, B, q, kc, vc, ref)
    torch.cuda.synchronize()
    assert plan.poll() == 0
    plan.close()
    got = torch.full(q.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    binding.forward_static(scales, H, k, B, q, kc, vc, got, share_cfg=share, rho=rho, radius=radius)
    torch.cuda.synchronize()
    g, r = got.double().cpu().numpy(), ref.double().cpu().numpy()
    assert np.isfinite(g).all()
    ma, rl = errors(g, r)
    assert ma <= MAX_ABS and rl <= REL_L2, (k, ma, rl)


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

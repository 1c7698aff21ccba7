"""Helpers shared by the GPU parity tests."""
import numpy as np
import torch

from oracle import litevar_oracle as orc
from paper_2411_17178_b200 import binding, build

MAX_ABS = 1e-2     # parity tolerance for bf16 inputs with fp32 accumulation: bf16 rounding of P and of the output
REL_L2 = 5e-3


def lib_ready():
    build.build()
    return binding.load()


def errors(got: np.ndarray, ref: np.ndarray):
    d = got.astype(np.float64) - ref
    return float(np.abs(d).max()), float(np.sqrt((d * d).sum()) / max(np.sqrt((ref * ref).sum()), 1e-300))


def assert_close(got, ref, what=""):
    ma, rl = errors(got, ref)
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    assert ma <= MAX_ABS and rl <= REL_L2, f"{what}: max-abs {ma:.3e} rel-L2 {rl:.3e}"
    return ma, rl


def run_forward(plan, step_k, B, Q, Kc, Vc, kernel=None, out=None):
    """Q/K/V host bf16 tensors -> device, one forward, output back as fp64 numpy."""
    if kernel is not None:
        plan.set_kernel(kernel)
    q, k, v = Q.cuda(), Kc.cuda(), Vc.cuda()
    if out is None:
        out = torch.full(q.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    plan.forward(step_k, B, q, k, v, out)
    torch.cuda.synchronize()
    assert plan.poll() == 0
    return out.double().cpu().numpy(), out


def oracle_radius(scales, rho=(1, 4), n_global=3):
    return orc.window_table(scales, rho=rho, n_global_scales=n_global)

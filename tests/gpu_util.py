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


def stratified_samples(plan, step_k, rows, n_heads, s_k, per_unit, rng, every=10):
    """(batch row, head, query) triples for the sampled parity checks at sizes the oracle cannot evaluate in full.

    Every (batch row, head) unit gets `per_unit` rows: the four grid corners, two edge mid-points and the grid
    centre in rotation, one row from each of the two heaviest and the two lightest query tiles of the plan (the
    first and the last CTAs of the launch order), and random rows.  Every `every`-th unit in addition gets one
    random valid row from EVERY query tile of the step, so that a fault confined to one tile, one CTA half or
    one position of the launch order is seen."""
    tiles = plan.export_tiles(step_k)
    geom, row_ptr = tiles["q_tile_geom"], tiles["row_ptr"]
    n_k = s_k * s_k
    weight = np.diff(row_ptr)
    order = np.argsort(-weight, kind="stable")
    extremes = list(order[:2]) + list(order[-2:])

    def row_of_tile(t):
        first, cols, stride, vr, vc = (int(x) for x in geom[t])
        r, c = int(rng.integers(0, vr)), int(rng.integers(0, vc))
        return first + r * stride + c

    fixed = [0, s_k - 1, n_k - s_k, n_k - 1, (s_k // 2) * s_k + s_k // 2, (s_k // 2) * s_k, s_k // 2]
    out = []
    for u in range(rows * n_heads):
        b, h = divmod(u, n_heads)
        qs = [fixed[u % len(fixed)], fixed[(u + 3) % len(fixed)]] + [row_of_tile(t) for t in extremes]
        if u % every == 0:
            qs += [row_of_tile(t) for t in range(len(geom))]
        while len(qs) < per_unit:
            qs.append(int(rng.integers(0, n_k)))
        out += [(b, h, int(q)) for q in qs]
    return out


def check_sampled(out, ref, samples, what):
    got = out.double().cpu().numpy() if hasattr(out, "double") else out
    g = np.stack([got[b, h, q] for b, h, q in samples])
    return assert_close(g, ref, what)

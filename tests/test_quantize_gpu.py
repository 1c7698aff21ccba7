"""8-bit Q/K/V (paper Section 4): the row quantiser kernel against the oracle, bit for bit, and the attention
on quantised Q/K/V against the oracle's attention on the oracle's dequantised tensors.

Codes, scales and zero points are decided in fp32 with the same sequence of IEEE operations on both sides, so
they must agree exactly; so must the dequantised bf16 rows."""
import numpy as np
import pytest
import torch

from oracle import litevar_oracle as orc
from paper_2411_17178_b200 import binding, workloads as wl
from tests.gpu_util import assert_close, errors, lib_ready

pytestmark = pytest.mark.gpu


def _rows(shape, seed, kind):
    g = torch.Generator().manual_seed(seed)
    x = torch.randn(*shape, generator=g, dtype=torch.float32)
    if kind == "offset":        # activations with a per-head offset and a few outliers, as after a projection
        x = x * 0.3 + torch.linspace(-2, 2, shape[1]).view(1, -1, 1, 1)
        x[..., 5] *= 9.0
    if kind == "ties":          # small integers: (x - z) / s hits exact ties
        x = torch.randint(-6, 7, shape, generator=g).float()
    return x.to(torch.bfloat16)


def _check_against_oracle(x, bits, got):
    out, codes, scale, zero = got
    c, s, z, deq = orc.quantize_rows(x.float().cpu().numpy(), bits)
    assert np.array_equal(scale.cpu().numpy(), s[..., 0])
    assert np.array_equal(zero.cpu().numpy(), z[..., 0])
    assert np.array_equal(codes.cpu().numpy().astype(np.int32), c)
    assert np.array_equal(out.float().cpu().numpy(), deq)


@pytest.mark.parametrize("kind", ["normal", "offset", "ties"])
@pytest.mark.parametrize("shape", [(1, 1, 1, 64), (2, 3, 5, 64), (4, 16, 680, 64), (3, 5, 1037, 64)])
def test_quantiser_matches_oracle_bit_for_bit(shape, kind):
    lib_ready()
    x = _rows(shape, 11 + shape[2], kind).cuda()
    _check_against_oracle(x, 8, binding.quantize_rows(x, 8, want_codes=True))


@pytest.mark.parametrize("bits", [2, 4, 6])
def test_quantiser_other_bit_widths(bits):
    lib_ready()
    x = _rows((2, 4, 91, 64), 3, "offset").cuda()
    _check_against_oracle(x, bits, binding.quantize_rows(x, bits, want_codes=True))


def test_quantiser_in_place_strided_and_degenerate_rows():
    lib_ready()
    # a [B, H, T, 64] view into a larger cache allocation: token stride 64, head stride of the full cache
    cache = _rows((2, 4, 300, 64), 5, "normal").cuda()
    view = cache[:, :, 40:140]
    before = cache.clone()
    want = orc.quantize_rows(view.float().cpu().numpy())[3]
    ret = binding.quantize_rows(view, out=view)
    assert ret.data_ptr() == view.data_ptr()
    assert np.array_equal(view.float().cpu().numpy(), want)
    assert torch.equal(cache[:, :, :40], before[:, :, :40]) and torch.equal(cache[:, :, 140:], before[:, :, 140:])
    # constant and all-zero rows
    const = torch.full((1, 2, 7, 64), 1.375, dtype=torch.bfloat16, device="cuda")
    const[0, 1] = 0
    out, codes, scale, zero = binding.quantize_rows(const, want_codes=True)
    assert torch.equal(out, const) and not codes.any() and not scale.any()
    assert torch.equal(zero[0, 0], torch.full((7,), 1.375, device="cuda"))


def test_quantiser_argument_errors():
    lib_ready()
    x = torch.zeros(1, 1, 4, 64, dtype=torch.bfloat16, device="cuda")
    for bits in (1, 9):
        with pytest.raises(binding.LitevarError) as e:
            binding.quantize_rows(x, bits)
        assert e.value.status == 1
    lib = binding.load()
    import ctypes
    s = binding._strides(x)
    assert lib.litevar_quantize_rows(None, ctypes.byref(s), 1, 1, 4, 64, 8, None, None, None, None, None, None) == 1
    assert lib.litevar_quantize_rows(x.data_ptr(), ctypes.byref(s), 1, 1, 4, 32, 8, None, None, None, None, None, None) == 2
    assert lib.litevar_quantize_rows(x.data_ptr() + 2, ctypes.byref(s), 1, 1, 4, 64, 8, None, None, None, None, None, None) == 1


def test_quantise_qkv_of_one_step_in_one_launch():
    """The step's Q and the cache rows appended at this step, in place; earlier cache rows are not touched."""
    lib_ready()
    scales, k, H, rows = wl.SCALES_256, 8, 3, 2
    off = orc.offsets(scales)
    n_k, L_k = orc.map_shape(scales, k)
    Q = _rows((rows, H, n_k, 64), 41, "offset")
    Kc = _rows((rows, H, L_k + 20, 64), 42, "offset")      # a cache with room beyond this step
    Vc = _rows((rows, H, L_k + 20, 64), 43, "normal")
    qd, kd, vd = Q.cuda(), Kc.cuda(), Vc.cuda()
    binding.quantize_qkv(qd, kd[:, :, off[k - 1]:L_k], vd[:, :, off[k - 1]:L_k])
    torch.cuda.synchronize()
    for dev, host, lo, hi in ((qd, Q, 0, n_k), (kd, Kc, off[k - 1], L_k), (vd, Vc, off[k - 1], L_k)):
        want = orc.quantize_rows(host[:, :, lo:hi].float().numpy())[3]
        assert np.array_equal(dev[:, :, lo:hi].float().cpu().numpy(), want)
        assert torch.equal(dev[:, :, :lo].cpu(), host[:, :, :lo]) and torch.equal(dev[:, :, hi:].cpu(), host[:, :, hi:])
    with pytest.raises(binding.LitevarError):
        binding.quantize_qkv(qd, kd[:, :, :4], vd[:, :, :4], bits=9)


@pytest.mark.parametrize("k", [4, 7, 10])
def test_attention_on_8bit_qkv(k):
    """QKV8 end to end at 256px: quantise Q and the cache rows on the device, run the windowed attention on the
    dequantised rows; the oracle does the same with its own quantiser and its fp64 attention."""
    lib_ready()
    w = wl.WORKLOADS[1]
    scales, H, B = w.scales, 4, 1
    n_k, L_k = orc.map_shape(scales, k)
    Q = _rows((2 * B, H, n_k, 64), 100 + k, "offset")
    Kc = _rows((2 * B, H, L_k, 64), 200 + k, "offset")
    Vc = _rows((2 * B, H, L_k, 64), 300 + k, "normal")
    tab = orc.window_table(scales)
    plan = binding.Plan(scales, n_heads=H)
    qd, kd, vd = (binding.quantize_rows(t.cuda()) for t in (Q, Kc, Vc))
    out = torch.full(qd.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    plan.forward(k, B, qd, kd, vd, out)
    torch.cuda.synchronize()
    assert plan.poll() == 0
    deq = [torch.from_numpy(orc.quantize_rows(t.float().numpy())[3]) for t in (Q, Kc, Vc)]
    ref = orc.attention_step(scales, k, tab[k - 1], *deq)
    assert_close(out.double().cpu().numpy(), ref, f"QKV8 step {k}")
    # the quantisation itself moves the result by far more than the parity tolerance (0.06 - 0.2 here), so the
    # check above does exercise it
    plain = orc.attention_step(scales, k, tab[k - 1], Q, Kc, Vc)
    assert 0.03 < np.abs(ref - plain).max() < 0.4
    plan.close()


def _cache8(t, rows_extra=0):
    """Quantise a bf16 cache tensor on the device: (codes, scale, zero, dequantised bf16)."""
    out, codes, scale, zero = binding.quantize_rows(t, want_codes=True)
    return codes, scale, zero, out


@pytest.mark.parametrize("scales,H,B,share,steps", [
    (wl.SCALES_256, 3, 1, True, (1, 3, 5, 7, 8, 9, 10)),      # small and large steps, shared
    (wl.SCALES_512, 2, 1, False, (7, 9, 10)),                 # several query tiles, long lists, unshared
    ((1, 2, 3, 4, 6, 9, 13, 18, 24), 2, 2, True, (8, 9)),     # ragged last query and key tiles
], ids=["256px", "512px", "ragged"])
def test_attention_reads_the_8bit_cache(scales, H, B, share, steps):
    """litevar_attn_forward_kv8: the attention kernel itself reads int8 codes, scales and zero points and widens
    them on the way into its shared-memory stages.  Its output must agree closely with the bf16 entry point run
    on the dequantised cache, and within the parity tolerance with the oracle's attention on the oracle's
    dequantised tensors.  The cache tensors are longer than L_k and their tail is poisoned."""
    lib_ready()
    K = len(scales)
    L = orc.map_shape(scales, K)[1]
    Kc = _rows((2 * B, H, L + 40, 64), 700 + K, "offset")
    Vc = _rows((2 * B, H, L + 40, 64), 800 + K, "normal")
    kc8, ks, kz, kdq = _cache8(Kc.cuda())
    vc8, vs, vz, vdq = _cache8(Vc.cuda())
    plan = binding.Plan(scales, n_heads=H, share_steps=[1] * K if share else None, tiling=binding.TILING_RASTER)
    tab = orc.window_table(scales)
    kdq_h = torch.from_numpy(orc.quantize_rows(Kc.float().numpy())[3])
    vdq_h = torch.from_numpy(orc.quantize_rows(Vc.float().numpy())[3])
    assert np.array_equal(kdq.float().cpu().numpy(), kdq_h.numpy())
    for k in steps:
        n_k, L_k = orc.map_shape(scales, k)
        Q = _rows((2 * B, H, n_k, 64), 900 + k, "normal")
        qd = binding.quantize_rows(Q.cuda())                  # 8-bit queries too (Section 4: Q, K and V)
        # rows beyond L_k must never reach the result: poison them in the 8-bit cache
        kc8p, ksp = kc8.clone(), ks.clone()
        kc8p[:, :, L_k:] = 127
        ksp[:, :, L_k:] = float("nan")
        want = torch.full(qd.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
        plan.set_kernel(binding.KERNEL_TCGEN05)
        plan.forward(k, B, qd, kdq, vdq, want)
        got = torch.full(qd.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
        plan.forward_kv8(k, B, qd, kc8p, ksp, kz, vc8, vs, vz, got)
        torch.cuda.synchronize()
        assert plan.poll() == 0
        # the widening rounds code * s + z once (a fused multiply-add on a shifted zero point) where the quantiser's
        # dequantised rows round product and sum separately: a few operands differ by one bf16 unit, so the two
        # outputs agree far inside the parity tolerance but not bit for bit
        ma, rl = errors(got.double().cpu().numpy(), want.double().cpu().numpy())
        assert ma <= 8e-3 and rl <= 3e-3, f"step {k}: 8-bit cache path against the bf16 path: {ma:.2e} {rl:.2e}"
        qdq_h = torch.from_numpy(orc.quantize_rows(Q.float().numpy())[3])
        ref = orc.attention_step(scales, k, tab[k - 1], qdq_h, kdq_h, vdq_h, share_cfg=share)
        assert_close(got.double().cpu().numpy(), ref, f"8-bit cache step {k}")
        # under AUTO the small steps read the 8-bit cache in the small-step kernel
        plan.set_kernel(binding.KERNEL_AUTO)
        got_auto = torch.full(qd.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
        plan.forward_kv8(k, B, qd, kc8p, ksp, kz, vc8, vs, vz, got_auto)
        torch.cuda.synchronize()
        assert plan.poll() == 0
        assert_close(got_auto.double().cpu().numpy(), ref, f"8-bit cache step {k}, kernel chosen by the plan")
        small = plan.step_kernel(k, B) == binding.KERNEL_SMALL
        assert small or torch.equal(got_auto.view(torch.int16), got.view(torch.int16))
        if share:
            assert torch.equal(got[:B].view(torch.int16), got[B:].view(torch.int16))
    plan.close()


def test_8bit_cache_argument_errors():
    lib_ready()
    scales = wl.SCALES_2K
    plan = binding.Plan(scales, n_heads=1)                    # patch tiles at the last steps
    q = torch.zeros(2, 1, 16384, 64, dtype=torch.bfloat16, device="cuda")
    c = torch.zeros(2, 1, 8, 64, dtype=torch.int8, device="cuda")       # never dereferenced
    z = torch.zeros(2, 1, 8, dtype=torch.float32, device="cuda")
    with pytest.raises(binding.LitevarError) as e:
        plan.forward_kv8(14, 1, q, c, z, z, c, z, z, q)
    assert e.value.status == 2
    plan.close()
    plan = binding.Plan((1, 2, 3, 4), n_heads=1)
    q = torch.zeros(2, 1, 16, 64, dtype=torch.bfloat16, device="cuda")
    c = torch.zeros(2, 1, 30, 64, dtype=torch.int8, device="cuda")
    z = torch.zeros(2, 1, 30, dtype=torch.float32, device="cuda")
    plan.forward_kv8(4, 1, q, c, z, z, c, z, z, q)                       # fine
    with pytest.raises(binding.LitevarError) as e:
        plan.forward_kv8(5, 1, q, c, z, z, c, z, z, q)
    assert e.value.status == 1
    lib = binding.load()
    import ctypes
    sq, sc, sr = binding._strides(q), binding._Strides(1920, 1920, 64), binding._Strides(30, 30, 1)
    bad = binding._Strides(1920, 1920, 72)                               # rows not on 16-byte boundaries
    args = lambda codes, srow: (plan._h, 4, 1, q.data_ptr(), ctypes.byref(sq), c.data_ptr(), z.data_ptr(), z.data_ptr(),
                                c.data_ptr(), z.data_ptr(), z.data_ptr(), ctypes.byref(codes), ctypes.byref(srow),
                                q.data_ptr(), ctypes.byref(sq), None)
    assert lib.litevar_attn_forward_kv8(*args(sc, sr)) == 0
    assert lib.litevar_attn_forward_kv8(*args(bad, sr)) == 1
    assert lib.litevar_attn_forward_kv8(*args(sc, binding._Strides(30, 30, 2))) == 1
    torch.cuda.synchronize()
    plan.close()

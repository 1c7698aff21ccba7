"""8-bit Q/K/V (paper Section 4): the row quantiser kernel against the oracle, bit for bit, and the attention
on quantised Q/K/V against the oracle's attention on the oracle's dequantised tensors.

Codes, scales and zero points are decided in fp32 with the same sequence of IEEE operations on both sides, so
they must agree exactly; so must the dequantised bf16 rows."""
import numpy as np
import pytest
import torch

from oracle import litevar_oracle as orc
from paper_2411_17178_b200 import binding, workloads as wl
from tests.gpu_util import assert_close, lib_ready

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

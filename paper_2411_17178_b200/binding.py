"""Thin ctypes binding of liblitevar.so: argument marshalling only.

Function names mirror the C ABI declared in ``include/litevar.h``.  Torch tensors are used as
device-memory handles (data pointer + strides) and for streams; every step of the attention
path runs in the library's own CUDA kernels.  There is no fallback: if the shared library has
not been built, loading raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liblitevar.so")

OK = 0
STATUS_NAMES = {0: "OK", 1: "INVALID_ARG", 2: "UNSUPPORTED", 3: "EMPTY_ROW", 4: "ARCH", 5: "OOM", 6: "CUDA",
                7: "DEVICE_TIMEOUT"}
WINDOW_SQUARE, WINDOW_BAND = 0, 1
KERNEL_AUTO, KERNEL_SIMT, KERNEL_TCGEN05, KERNEL_SMALL, KERNEL_TCGEN05_WS = 0, 1, 2, 3, 4
TILING_AUTO, TILING_RASTER, TILING_PATCH = 0, 1, 2

EXPORTS = (
    "litevar_attn_plan", "litevar_attn_forward", "litevar_attn_forward_kv8", "litevar_attn_forward_static",
    "litevar_calibrate_windows",
    "litevar_quantize_rows", "litevar_quantize_qkv",
    "litevar_plan_stats", "litevar_plan_tile_counts",
    "litevar_plan_export_tiles", "litevar_plan_export_bounds", "litevar_plan_materialize_mask",
    "litevar_plan_poll_device_status", "litevar_plan_set_kernel", "litevar_plan_step_kernel", "litevar_plan_destroy",
    "litevar_status_string",
)


class LitevarError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)}")


class _Window(ctypes.Structure):
    _fields_ = [("shape", ctypes.c_int32), ("n_global_scales", ctypes.c_int32),
                ("rho_num", ctypes.c_int32), ("rho_den", ctypes.c_int32),
                ("radius", ctypes.POINTER(ctypes.c_int32)), ("n_sets", ctypes.c_int32),
                ("head_to_set", ctypes.POINTER(ctypes.c_int32)), ("tiling", ctypes.c_int32)]


class _Share(ctypes.Structure):
    _fields_ = [("share_step", ctypes.POINTER(ctypes.c_uint8))]


class _Strides(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int64), ("head", ctypes.c_int64), ("token", ctypes.c_int64)]


_lib = None


def load() -> ctypes.CDLL:
    """Load the C-ABI library; raises if it is missing (there is no other compute path)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            f"{LIB_PATH} not found: build it with `python -m paper_2411_17178_b200.build` "
            "(needs nvcc; the library has no CPU or PyTorch fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    P, I32, I64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
    lib.litevar_attn_plan.restype = ctypes.c_int
    lib.litevar_attn_plan.argtypes = [ctypes.POINTER(I32), I32, I32, I32, ctypes.c_float,
                                      ctypes.POINTER(_Window), ctypes.POINTER(_Share), P, ctypes.POINTER(P)]
    lib.litevar_attn_forward.restype = ctypes.c_int
    lib.litevar_attn_forward.argtypes = [P, I32, I32, P, ctypes.POINTER(_Strides), P, ctypes.POINTER(_Strides),
                                         P, ctypes.POINTER(_Strides), P, ctypes.POINTER(_Strides), P]
    lib.litevar_attn_forward_kv8.restype = ctypes.c_int
    lib.litevar_attn_forward_kv8.argtypes = [P, I32, I32, P, ctypes.POINTER(_Strides), P, P, P, P, P, P,
                                             ctypes.POINTER(_Strides), ctypes.POINTER(_Strides), P,
                                             ctypes.POINTER(_Strides), P]
    lib.litevar_attn_forward_static.restype = ctypes.c_int
    lib.litevar_attn_forward_static.argtypes = [ctypes.POINTER(I32), I32, I32, I32, ctypes.c_float,
                                                ctypes.POINTER(_Window), I32, I32, I32,
                                                P, ctypes.POINTER(_Strides), P, ctypes.POINTER(_Strides),
                                                P, ctypes.POINTER(_Strides), P, ctypes.POINTER(_Strides), P]
    lib.litevar_calibrate_windows.restype = ctypes.c_int
    lib.litevar_calibrate_windows.argtypes = [ctypes.POINTER(I32), I32, I32, I32, P, I64, ctypes.c_double, P, P, P]
    lib.litevar_quantize_rows.restype = ctypes.c_int
    lib.litevar_quantize_rows.argtypes = [P, ctypes.POINTER(_Strides), I32, I32, I32, I32, I32, P,
                                          ctypes.POINTER(_Strides), P, P, P, P]
    lib.litevar_quantize_qkv.restype = ctypes.c_int
    lib.litevar_quantize_qkv.argtypes = [P, ctypes.POINTER(_Strides), I32, P, ctypes.POINTER(_Strides), P,
                                         ctypes.POINTER(_Strides), I32, I32, I32, I32, I32, P]
    lib.litevar_plan_stats.restype = ctypes.c_int
    lib.litevar_plan_stats.argtypes = [P, I32, I32] + [ctypes.POINTER(I64)] * 4
    lib.litevar_plan_tile_counts.restype = ctypes.c_int
    lib.litevar_plan_tile_counts.argtypes = [P, I32, I32] + [ctypes.POINTER(I32)] * 3
    lib.litevar_plan_export_tiles.restype = ctypes.c_int
    lib.litevar_plan_export_tiles.argtypes = [P, I32, I32, P, P, P, P, P]
    lib.litevar_plan_export_bounds.restype = ctypes.c_int
    lib.litevar_plan_export_bounds.argtypes = [P, I32, I32, P, P]
    lib.litevar_plan_materialize_mask.restype = ctypes.c_int
    lib.litevar_plan_materialize_mask.argtypes = [P, I32, I32, P, P]
    lib.litevar_plan_poll_device_status.restype = ctypes.c_int
    lib.litevar_plan_poll_device_status.argtypes = [P]
    lib.litevar_plan_set_kernel.restype = ctypes.c_int
    lib.litevar_plan_set_kernel.argtypes = [P, I32]
    lib.litevar_plan_step_kernel.restype = ctypes.c_int
    lib.litevar_plan_step_kernel.argtypes = [P, I32, I32, ctypes.POINTER(I32)]
    lib.litevar_plan_destroy.restype = None
    lib.litevar_plan_destroy.argtypes = [P]
    lib.litevar_status_string.restype = ctypes.c_char_p
    lib.litevar_status_string.argtypes = [ctypes.c_int]
    _lib = lib
    return lib


def _check(status: int, where: str) -> None:
    if status != OK:
        raise LitevarError(status, where)


def _i32_array(values) -> ctypes.Array:
    vals = [int(v) for v in values]
    return (ctypes.c_int32 * len(vals))(*vals)


def _stream_ptr(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return getattr(stream, "cuda_stream", stream)


def _current_raw_stream(device_index) -> int:
    """cudaStream_t of torch's current stream on that device, without building a Stream object."""
    import torch
    try:
        return torch._C._cuda_getCurrentRawStream(device_index if device_index is not None else torch.cuda.current_device())
    except AttributeError:
        return torch.cuda.current_stream().cuda_stream


def _strides(t) -> _Strides:
    assert t.dim() == 4 and t.stride(3) == 1, "expected [2B, H, tokens, 64] with contiguous head_dim"
    return _Strides(t.stride(0), t.stride(1), t.stride(2))


class Plan:
    """Owner of a ``litevar_plan_t*`` (see litevar_attn_plan)."""

    def __init__(self, scales: Sequence[int], n_heads: int, head_dim: int = 64, sm_scale: float = 0.0,
                 shape: int = WINDOW_SQUARE, n_global_scales: int = 3, rho=(1, 4), radius=None,
                 n_sets: int = 1, head_to_set=None, share_steps=None, stream=None, tiling: int = TILING_AUTO):
        lib = load()
        self._lib = lib
        self.scales = tuple(int(s) for s in scales)
        self.n_heads = int(n_heads)
        self.n_sets = int(n_sets)
        K = len(self.scales)
        win = _Window()
        win.shape, win.n_global_scales = int(shape), int(n_global_scales)
        win.rho_num, win.rho_den = int(rho[0]), int(rho[1])
        win.n_sets = self.n_sets
        win.tiling = int(tiling)
        keep = []
        if radius is not None:
            arr = np.ascontiguousarray(np.asarray(radius, dtype=np.int32).reshape(self.n_sets, K, K))
            keep.append(arr)
            win.radius = arr.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))
        if head_to_set is not None:
            h2s = _i32_array(head_to_set)
            keep.append(h2s)
            win.head_to_set = ctypes.cast(h2s, ctypes.POINTER(ctypes.c_int32))
        share = _Share()
        if share_steps is not None:
            flags = (ctypes.c_uint8 * K)(*[1 if s else 0 for s in share_steps])
            keep.append(flags)
            share.share_step = ctypes.cast(flags, ctypes.POINTER(ctypes.c_uint8))
        handle = ctypes.c_void_p()
        st = lib.litevar_attn_plan(_i32_array(self.scales), K, self.n_heads, int(head_dim), float(sm_scale),
                                   ctypes.byref(win), ctypes.byref(share), _stream_ptr(stream),
                                   ctypes.byref(handle))
        _check(st, "litevar_attn_plan")
        self._h = handle
        self._strides4 = tuple(_Strides(0, 0, 0) for _ in range(4))
        self._strides4_ref = tuple(ctypes.byref(x) for x in self._strides4)

    def close(self) -> None:
        if getattr(self, "_h", None):
            self._lib.litevar_plan_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- forward ---------------------------------------------------------------------------
    def forward(self, step_k: int, batch_pairs: int, q, k_cache, v_cache, out, stream=None) -> None:
        """litevar_attn_forward on torch CUDA tensors (bf16, [2B, H, tokens, 64]).

        The marshalling is kept short (it is most of an eager call's host time): the four stride structs live
        in the plan and are refilled, so one plan must not be driven from several Python threads at once."""
        sq, sk, sv, so = self._strides4
        a = q.stride()
        sq.batch, sq.head, sq.token = a[0], a[1], a[2]
        b = k_cache.stride()
        sk.batch, sk.head, sk.token = b[0], b[1], b[2]
        c = v_cache.stride()
        sv.batch, sv.head, sv.token = c[0], c[1], c[2]
        d = out.stride()
        so.batch, so.head, so.token = d[0], d[1], d[2]
        if a[3] != 1 or b[3] != 1 or c[3] != 1 or d[3] != 1:
            raise ValueError("expected [2B, H, tokens, 64] tensors with contiguous head_dim")
        if stream is None:
            stream_ptr = _current_raw_stream(q.device.index)
        else:
            stream_ptr = getattr(stream, "cuda_stream", stream)
        st = self._lib.litevar_attn_forward(self._h, step_k, batch_pairs, q.data_ptr(), self._strides4_ref[0],
                                            k_cache.data_ptr(), self._strides4_ref[1], v_cache.data_ptr(),
                                            self._strides4_ref[2], out.data_ptr(), self._strides4_ref[3], stream_ptr)
        if st != 0:
            _check(st, "litevar_attn_forward")

    def forward_kv8(self, step_k: int, batch_pairs: int, q, k_codes, k_scale, k_zero, v_codes, v_scale, v_zero, out,
                    stream=None) -> None:
        """litevar_attn_forward_kv8 on torch CUDA tensors: q/out bf16 [2B, H, n_k, 64]; codes int8 [2B, H, rows, 64]
        (K and V with the same strides); scales and zero points fp32 [2B, H, rows] (all four with the same strides)."""
        assert k_codes.stride() == v_codes.stride() and k_codes.stride(3) == 1
        assert k_scale.stride() == k_zero.stride() == v_scale.stride() == v_zero.stride() and k_scale.stride(2) == 1
        sc = _Strides(k_codes.stride(0), k_codes.stride(1), k_codes.stride(2))
        sr = _Strides(k_scale.stride(0), k_scale.stride(1), 1)
        stream_ptr = _current_raw_stream(q.device.index) if stream is None else getattr(stream, "cuda_stream", stream)
        st = self._lib.litevar_attn_forward_kv8(
            self._h, int(step_k), int(batch_pairs), q.data_ptr(), ctypes.byref(_strides(q)), k_codes.data_ptr(),
            k_scale.data_ptr(), k_zero.data_ptr(), v_codes.data_ptr(), v_scale.data_ptr(), v_zero.data_ptr(),
            ctypes.byref(sc), ctypes.byref(sr), out.data_ptr(), ctypes.byref(_strides(out)), stream_ptr)
        _check(st, "litevar_attn_forward_kv8")

    def forward_raw(self, step_k, batch_pairs, q_ptr, q_str, k_ptr, k_str, v_ptr, v_str, o_ptr, o_str,
                    stream_ptr) -> int:
        """Unchecked call with raw pointers and (batch, head, token) stride triples; returns the status."""
        return self._lib.litevar_attn_forward(
            self._h, int(step_k), int(batch_pairs), q_ptr, ctypes.byref(_Strides(*q_str)), k_ptr,
            ctypes.byref(_Strides(*k_str)), v_ptr, ctypes.byref(_Strides(*v_str)), o_ptr,
            ctypes.byref(_Strides(*o_str)), stream_ptr)

    # -- introspection ---------------------------------------------------------------------
    def stats(self, step_k: int, set_index: int = 0) -> dict:
        vals = [ctypes.c_int64() for _ in range(4)]
        _check(self._lib.litevar_plan_stats(self._h, int(step_k), int(set_index), *[ctypes.byref(v) for v in vals]),
               "litevar_plan_stats")
        return dict(zip(("live_entries", "live_tiles", "full_tiles", "partial_tiles"), (v.value for v in vals)))

    def tile_counts(self, step_k: int, set_index: int = 0):
        vals = [ctypes.c_int32() for _ in range(3)]
        _check(self._lib.litevar_plan_tile_counts(self._h, int(step_k), int(set_index),
                                                  *[ctypes.byref(v) for v in vals]), "litevar_plan_tile_counts")
        return tuple(v.value for v in vals)

    def export_tiles(self, step_k: int, set_index: int = 0) -> dict:
        nq, nk, npairs = self.tile_counts(step_k, set_index)
        qg = np.zeros((nq, 5), np.int32)
        kg = np.zeros((nk, 5), np.int32)
        rp = np.zeros(nq + 1, np.int32)
        pk = np.zeros(max(npairs, 1), np.int32)
        pf = np.zeros(max(npairs, 1), np.uint8)
        _check(self._lib.litevar_plan_export_tiles(self._h, int(step_k), int(set_index), qg.ctypes.data,
                                                   kg.ctypes.data, rp.ctypes.data, pk.ctypes.data, pf.ctypes.data),
               "litevar_plan_export_tiles")
        return dict(q_tile_geom=qg, key_tile_geom=kg, row_ptr=rp, pair_key_tile=pk[:npairs],
                    pair_is_full=pf[:npairs])

    def export_bounds(self, step_k: int, set_index: int = 0):
        K = len(self.scales)
        s_k = self.scales[step_k - 1]
        rad = np.zeros(K, np.int32)
        bnd = np.zeros((step_k, s_k, 2), np.int32)
        _check(self._lib.litevar_plan_export_bounds(self._h, int(step_k), int(set_index), rad.ctypes.data,
                                                    bnd.ctypes.data), "litevar_plan_export_bounds")
        return rad, bnd

    def materialize_mask(self, step_k: int, set_index: int = 0, stream=None):
        """Dense boolean mask [n_k, L_k] (numpy) expanded on the device from the tile plan."""
        import torch
        s_k = self.scales[step_k - 1]
        n_k = s_k * s_k
        L_k = sum(s * s for s in self.scales[:step_k])
        words = (L_k + 31) // 32
        bits = torch.empty((n_k, words), dtype=torch.int32, device="cuda")
        _check(self._lib.litevar_plan_materialize_mask(self._h, int(step_k), int(set_index), bits.data_ptr(),
                                                       _stream_ptr(stream)), "litevar_plan_materialize_mask")
        torch.cuda.synchronize()
        w = bits.cpu().numpy().view(np.uint32)
        out = np.unpackbits(w.view(np.uint8), axis=1, bitorder="little")[:, :L_k].astype(bool)
        return out

    def poll(self) -> int:
        return self._lib.litevar_plan_poll_device_status(self._h)

    def set_kernel(self, kernel: int) -> None:
        _check(self._lib.litevar_plan_set_kernel(self._h, int(kernel)), "litevar_plan_set_kernel")

    def step_kernel(self, step_k: int, batch_pairs: int = 1) -> int:
        """KERNEL_SIMT, KERNEL_TCGEN05 or KERNEL_SMALL: what a forward of this step with that batch launches."""
        out = ctypes.c_int32(0)
        _check(self._lib.litevar_plan_step_kernel(self._h, int(step_k), int(batch_pairs), ctypes.byref(out)),
               "litevar_plan_step_kernel")
        return int(out.value)


STATIC_MAX_PAIRS = 2048


def forward_static(scales: Sequence[int], n_heads: int, step_k: int, batch_pairs: int, q, k_cache, v_cache, out,
                   share_cfg: bool = False, head_dim: int = 64, sm_scale: float = 0.0, shape: int = WINDOW_SQUARE,
                   n_global_scales: int = 3, rho=(1, 4), radius=None, stream=None) -> None:
    """litevar_attn_forward_static: step-k attention for callers that must not allocate device memory.

    No plan object: the step's tile plan is rebuilt on the device, inside a fixed array that belongs to
    the library, on every call.  Steps with more than STATIC_MAX_PAIRS candidate tile pairs are refused.
    Calls share that array, so keep them on one stream."""
    lib = load()
    K = len(scales)
    win = _Window()
    win.shape, win.n_global_scales = int(shape), int(n_global_scales)
    win.rho_num, win.rho_den = int(rho[0]), int(rho[1])
    win.n_sets = 1
    keep = None
    if radius is not None:
        keep = np.ascontiguousarray(np.asarray(radius, dtype=np.int32).reshape(K, K))
        win.radius = keep.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))
    st = lib.litevar_attn_forward_static(
        _i32_array(scales), K, int(n_heads), int(head_dim), float(sm_scale), ctypes.byref(win),
        1 if share_cfg else 0, int(step_k), int(batch_pairs),
        q.data_ptr(), ctypes.byref(_strides(q)), k_cache.data_ptr(), ctypes.byref(_strides(k_cache)),
        v_cache.data_ptr(), ctypes.byref(_strides(v_cache)), out.data_ptr(), ctypes.byref(_strides(out)),
        _stream_ptr(stream))
    if st == 2:
        raise LitevarError(st, "litevar_attn_forward_static (head_dim must be 64, one window set, and the step "
                               f"may have at most {STATIC_MAX_PAIRS} candidate tile pairs)")
    _check(st, "litevar_attn_forward_static")


def calibrate_windows(scales: Sequence[int], step_k: int, maps, r0: float, n_global_scales: int = 3,
                      want_ratio: bool = False, stream=None):
    """litevar_calibrate_windows on a CUDA float32 tensor [n_maps, n_k, L_k]; returns the radius row
    (numpy int32 [n_scales]) and, if asked, the R_w curves [n_scales, 256]."""
    lib = load()
    K = len(scales)
    assert maps.is_cuda and maps.dtype.is_floating_point and maps.element_size() == 4 and maps.is_contiguous()
    rad = np.zeros(K, np.int32)
    ratio = np.zeros((K, 256), np.float64) if want_ratio else None
    st = lib.litevar_calibrate_windows(_i32_array(scales), K, int(step_k), int(n_global_scales), maps.data_ptr(),
                                       int(maps.shape[0]), float(r0), rad.ctypes.data,
                                       ratio.ctypes.data if want_ratio else None, _stream_ptr(stream))
    _check(st, "litevar_calibrate_windows")
    return (rad, ratio) if want_ratio else rad


def quantize_rows(x, bits: int = 8, out=None, want_codes: bool = False, stream=None):
    """litevar_quantize_rows on a CUDA bf16 tensor [batch, heads, tokens, 64] (last dimension contiguous).
    Writes the dequantised rows to `out` (bf16, same shape; `x` itself for in place; a new tensor when None)
    and returns it, or (out, codes int8, scale fp32, zero fp32) when `want_codes`."""
    import torch
    lib = load()
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.dim() == 4 and x.stride(3) == 1
    if out is None:
        out = torch.empty(x.shape, dtype=torch.bfloat16, device=x.device)
    assert out.is_cuda and out.dtype == torch.bfloat16 and out.shape == x.shape and out.stride(3) == 1
    B, H, T, D = x.shape
    codes = scale = zero = None
    if want_codes:
        codes = torch.empty((B, H, T, D), dtype=torch.int8, device=x.device)
        scale = torch.empty((B, H, T), dtype=torch.float32, device=x.device)
        zero = torch.empty((B, H, T), dtype=torch.float32, device=x.device)
    st = lib.litevar_quantize_rows(x.data_ptr(), ctypes.byref(_strides(x)), B, H, T, D, int(bits), out.data_ptr(),
                                   ctypes.byref(_strides(out)), codes.data_ptr() if want_codes else None,
                                   scale.data_ptr() if want_codes else None,
                                   zero.data_ptr() if want_codes else None, _stream_ptr(stream))
    _check(st, "litevar_quantize_rows")
    return (out, codes, scale, zero) if want_codes else out


def quantize_qkv(q, k_new, v_new, bits: int = 8, stream=None) -> None:
    """litevar_quantize_qkv: quantise-dequantise, in place and in one launch, the step's Q [batch, heads, n_k, 64]
    and the appended cache rows k_new, v_new [batch, heads, n_new, 64] (views into the caches)."""
    lib = load()
    B, H, Tq, D = q.shape
    assert k_new.shape == v_new.shape and k_new.shape[:2] == (B, H) and k_new.shape[3] == D
    st = lib.litevar_quantize_qkv(q.data_ptr(), ctypes.byref(_strides(q)), Tq, k_new.data_ptr(),
                                  ctypes.byref(_strides(k_new)), v_new.data_ptr(), ctypes.byref(_strides(v_new)),
                                  int(k_new.shape[2]), B, H, D, int(bits), _stream_ptr(stream))
    _check(st, "litevar_quantize_qkv")


def status_string(status: int) -> str:
    return load().litevar_status_string(int(status)).decode()

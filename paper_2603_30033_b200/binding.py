"""Thin ctypes binding of libtucker_attn.so (the C ABI declared in include/tucker_attn.h).

Only argument marshalling happens here: tensors are checked for device / dtype / contiguity,
their pointers and the current CUDA stream are handed to the library, and every step of the
computation runs in the library's kernels.  torch is used for device memory and streams
only.  If the library has not been built, loading raises; there is no fallback.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

_HERE = os.path.dirname(os.path.abspath(__file__))
# TUCKER_ATTN_LIB=checked selects the twin built with -DTA_BOUNDS_CHECK (device-side range checks on every
# global index, reported through the device error word); anything else, or nothing, the normal library.
LIB_PATH = os.path.join(_HERE, "libtucker_attn_checked.so" if os.environ.get("TUCKER_ATTN_LIB") == "checked"
                        else "libtucker_attn.so")

TA_OK = 0
TA_DTYPE_F32, TA_DTYPE_BF16 = 0, 1
TA_FLAG_FORCE_GENERIC = 1
TA_FLAG_FMA_ATTENTION, TA_FLAG_SEPARATE_QUERIES, TA_FLAG_SEPARATE_OUTPUT_GEMMS = 0x200, 0x400, 0x800
TA_DEVERR_WAIT_TIMEOUT, TA_DEVERR_BAD_CACHE_LEN, TA_DEVERR_BAD_INDEX = 1, 2, 4

EXPORTS = (
    "tucker_attn_fwd_workspace_bytes", "tucker_attn_decode_workspace_bytes", "tucker_attn_fwd",
    "tucker_attn_decode", "tucker_attn_status_string", "tucker_attn_last_device_error",
    "tucker_attn_last_path", "tucker_attn_last_launch_count", "tucker_attn_set_profile_events",
    "tucker_attn_decode_static", "tucker_attn_selftest_wait_timeout", "tucker_attn_sync_status",
    "tucker_attn_bounds_checked",
    "tucker_pack_gqa", "tucker_pack_mha", "tucker_pack_mla",
    "tucker_hosvd_workspace_bytes", "tucker_hosvd_init", "tucker_mha_weight_tensors", "tucker_probe_plane_mix", "tucker_probe_mma_rate",
)
TA_STATIC_SCRATCH_BYTES = 16 << 20


class TuckerAttnDesc(ctypes.Structure):
    """Mirror of `tucker_attn_desc`."""
    _fields_ = [
        ("B", ctypes.c_int32), ("N", ctypes.c_int32), ("d_model", ctypes.c_int32), ("n_H", ctypes.c_int32),
        ("r1", ctypes.c_int32), ("r2", ctypes.c_int32), ("r3", ctypes.c_int32),
        ("t1", ctypes.c_int32), ("t2", ctypes.c_int32), ("t3", ctypes.c_int32),
        ("causal", ctypes.c_int32), ("rope", ctypes.c_int32), ("rope_base", ctypes.c_float),
        ("pos0", ctypes.c_int32), ("scale", ctypes.c_float), ("dtype", ctypes.c_int32),
        ("flags", ctypes.c_int32),
    ]


class TuckerAttnError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where} failed: {status_string(status)} ({status})")


_lib = None


def load_library() -> ctypes.CDLL:
    """Loads the CUDA library; raises if it has not been built (no CPU fallback exists)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2603_30033_b200.build` "
            "(needs nvcc); this package has no fallback path")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_size_t
    dp = ctypes.POINTER(TuckerAttnDesc)
    lib.tucker_attn_fwd_workspace_bytes.restype = sz
    lib.tucker_attn_fwd_workspace_bytes.argtypes = [dp]
    lib.tucker_attn_decode_workspace_bytes.restype = sz
    lib.tucker_attn_decode_workspace_bytes.argtypes = [dp, i32]
    lib.tucker_attn_fwd.restype = ctypes.c_int
    lib.tucker_attn_fwd.argtypes = [dp] + [vp] * 12 + [i32, vp, sz, vp]
    lib.tucker_attn_decode.restype = ctypes.c_int
    lib.tucker_attn_decode.argtypes = [dp] + [vp] * 11 + [i32, vp, i32, vp, vp, sz, vp]
    lib.tucker_attn_decode_static.restype = ctypes.c_int
    lib.tucker_attn_decode_static.argtypes = [dp] + [vp] * 11 + [i32, vp, i32, vp, vp]
    lib.tucker_attn_status_string.restype = ctypes.c_char_p
    lib.tucker_attn_status_string.argtypes = [ctypes.c_int]
    lib.tucker_attn_last_device_error.restype = ctypes.c_int
    lib.tucker_attn_last_device_error.argtypes = [vp]
    lib.tucker_attn_sync_status.restype = ctypes.c_int
    lib.tucker_attn_sync_status.argtypes = [vp]
    lib.tucker_attn_bounds_checked.restype = ctypes.c_int
    lib.tucker_attn_last_path.restype = ctypes.c_int
    lib.tucker_attn_last_launch_count.restype = ctypes.c_int
    lib.tucker_attn_set_profile_events.restype = ctypes.c_int
    lib.tucker_attn_set_profile_events.argtypes = [vp, vp]
    lib.tucker_attn_selftest_wait_timeout.restype = ctypes.c_int
    lib.tucker_attn_selftest_wait_timeout.argtypes = [i32, vp, vp]
    lib.tucker_pack_gqa.restype = ctypes.c_int
    lib.tucker_pack_gqa.argtypes = [i32] * 4 + [vp] * 13
    lib.tucker_pack_mha.restype = ctypes.c_int
    lib.tucker_pack_mha.argtypes = [i32] * 3 + [vp] * 13
    lib.tucker_pack_mla.restype = ctypes.c_int
    lib.tucker_pack_mla.argtypes = [i32] * 5 + [vp] * 16
    lib.tucker_hosvd_workspace_bytes.restype = sz
    lib.tucker_hosvd_workspace_bytes.argtypes = [i32] * 4
    lib.tucker_hosvd_init.restype = ctypes.c_int
    lib.tucker_hosvd_init.argtypes = [i32] * 5 + [vp] * 7 + [sz, vp]
    lib.tucker_mha_weight_tensors.restype = ctypes.c_int
    lib.tucker_mha_weight_tensors.argtypes = [i32] * 2 + [vp] * 7
    lib.tucker_probe_mma_rate.restype = ctypes.c_int
    lib.tucker_probe_mma_rate.argtypes = [i32] * 4 + [vp] * 2
    lib.tucker_probe_plane_mix.restype = ctypes.c_int
    lib.tucker_probe_plane_mix.argtypes = [i32] * 3 + [vp] * 4
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load_library().tucker_attn_status_string(int(status)).decode()


def _torch():
    import torch
    return torch


def _dtype_code(t) -> int:
    torch = _torch()
    if t.dtype == torch.float32:
        return TA_DTYPE_F32
    if t.dtype == torch.bfloat16:
        return TA_DTYPE_BF16
    raise TypeError(f"unsupported dtype {t.dtype}; use float32 or bfloat16")


def _check(t, name, shape, dtype, device):
    if t.device != device or not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor on {device}")
    if t.dtype != dtype:
        raise TypeError(f"{name} has dtype {t.dtype}, expected {dtype}")
    if tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name} has shape {tuple(t.shape)}, expected {tuple(shape)}")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")


def make_desc(*, B, N, d_model, n_H, r, t, causal, rope, rope_base=10000.0, pos0=0, scale=0.0,
              dtype=TA_DTYPE_BF16, flags=0) -> TuckerAttnDesc:
    return TuckerAttnDesc(int(B), int(N), int(d_model), int(n_H), int(r[0]), int(r[1]), int(r[2]),
                          int(t[0]), int(t[1]), int(t[2]), int(bool(causal)), int(bool(rope)),
                          float(rope_base), int(pos0), float(scale), int(dtype), int(flags))


def fwd_workspace_bytes(desc: TuckerAttnDesc) -> int:
    return int(load_library().tucker_attn_fwd_workspace_bytes(ctypes.byref(desc)))


def decode_workspace_bytes(desc: TuckerAttnDesc, Lmax: int) -> int:
    return int(load_library().tucker_attn_decode_workspace_bytes(ctypes.byref(desc), int(Lmax)))


def alloc_workspace(nbytes: int, device):
    """Device scratch buffer (256-byte aligned by the torch allocator)."""
    torch = _torch()
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def _stream_ptr(device) -> int:
    return int(_torch().cuda.current_stream(device).cuda_stream)


def _weights_check(w, d_model, n_H, dtype, device):
    C, U1, U2, U3, Ct, Ut1, Ut2, Ut3 = w
    if C.dim() != 3 or Ct.dim() != 3:
        raise ValueError("cores must be 3-way tensors")
    r = tuple(C.shape)
    t = tuple(Ct.shape)
    _check(C, "C", r, dtype, device)
    _check(U1, "U1", (n_H, r[0]), dtype, device)
    _check(U2, "U2", (d_model, r[1]), dtype, device)
    _check(U3, "U3", (d_model, r[2]), dtype, device)
    _check(Ct, "Ct", t, dtype, device)
    _check(Ut1, "Ut1", (n_H, t[0]), dtype, device)
    _check(Ut2, "Ut2", (d_model, t[1]), dtype, device)
    _check(Ut3, "Ut3", (d_model, t[2]), dtype, device)
    return r, t


def tucker_attn_fwd(X, C, U1, U2, U3, Ct, Ut1, Ut2, Ut3, *, n_H: int, causal: bool, rope: bool,
                    rope_base: float = 10000.0, pos0: int = 0, scale: float = 0.0, out=None,
                    Kcache=None, Vcache=None, workspace=None, flags: int = 0):
    """Prefill forward (same name and argument meaning as the C entry point).  X [B, N, d];
    returns Y [B, N, d].  Kcache [B, Lmax, r3] / Vcache [B, Lmax, t3], when given, receive the
    rotated latent keys and the latent values in rows 0..N-1."""
    torch = _torch()
    lib = load_library()
    if X.dim() != 3:
        raise ValueError("X must be [B, N, d_model]")
    B, N, d = X.shape
    dev, dt = X.device, X.dtype
    _check(X, "X", (B, N, d), dt, dev)
    r, t = _weights_check((C, U1, U2, U3, Ct, Ut1, Ut2, Ut3), d, n_H, dt, dev)
    desc = make_desc(B=B, N=N, d_model=d, n_H=n_H, r=r, t=t, causal=causal, rope=rope, rope_base=rope_base,
                     pos0=pos0, scale=scale, dtype=_dtype_code(X), flags=flags)
    if out is None:
        out = torch.empty_like(X)
    _check(out, "out", (B, N, d), dt, dev)
    Lmax = 0
    kp = vp = None
    if (Kcache is None) != (Vcache is None):
        raise ValueError("pass both caches or neither")
    if Kcache is not None:
        Lmax = Kcache.shape[1]
        _check(Kcache, "Kcache", (B, Lmax, r[2]), dt, dev)
        _check(Vcache, "Vcache", (B, Lmax, t[2]), dt, dev)
        kp, vp = Kcache.data_ptr(), Vcache.data_ptr()
    need = lib.tucker_attn_fwd_workspace_bytes(ctypes.byref(desc))
    if workspace is None:
        workspace = alloc_workspace(need, dev)
    with torch.cuda.device(dev):
        rc = lib.tucker_attn_fwd(ctypes.byref(desc), X.data_ptr(), C.data_ptr(), U1.data_ptr(), U2.data_ptr(),
                                 U3.data_ptr(), Ct.data_ptr(), Ut1.data_ptr(), Ut2.data_ptr(), Ut3.data_ptr(),
                                 out.data_ptr(), kp, vp, int(Lmax), workspace.data_ptr(), workspace.numel(),
                                 _stream_ptr(dev))
    if rc != TA_OK:
        raise TuckerAttnError(rc, "tucker_attn_fwd")
    return out


def tucker_attn_decode(x, C, U1, U2, U3, Ct, Ut1, Ut2, Ut3, Kcache, Vcache, cache_len, *, n_H: int,
                       rope: bool, rope_base: float = 10000.0, scale: float = 0.0, append: bool = True,
                       out=None, workspace=None, flags: int = 0):
    """One cached decode step (same name and argument meaning as the C entry point).
    x [B, d]; Kcache [B, Lmax, r3] (rotated keys); Vcache [B, Lmax, t3]; cache_len int32 [B] on
    the device.  Returns y [B, d]."""
    torch = _torch()
    lib = load_library()
    if x.dim() != 2:
        raise ValueError("x must be [B, d_model]")
    B, d = x.shape
    dev, dt = x.device, x.dtype
    _check(x, "x", (B, d), dt, dev)
    r, t = _weights_check((C, U1, U2, U3, Ct, Ut1, Ut2, Ut3), d, n_H, dt, dev)
    Lmax = Kcache.shape[1]
    _check(Kcache, "Kcache", (B, Lmax, r[2]), dt, dev)
    _check(Vcache, "Vcache", (B, Lmax, t[2]), dt, dev)
    _check(cache_len, "cache_len", (B,), torch.int32, dev)
    desc = make_desc(B=B, N=1, d_model=d, n_H=n_H, r=r, t=t, causal=True, rope=rope, rope_base=rope_base,
                     pos0=0, scale=scale, dtype=_dtype_code(x), flags=flags)
    if out is None:
        out = torch.empty_like(x)
    _check(out, "out", (B, d), dt, dev)
    need = lib.tucker_attn_decode_workspace_bytes(ctypes.byref(desc), int(Lmax))
    if workspace is None:
        workspace = alloc_workspace(need, dev)
    with torch.cuda.device(dev):
        rc = lib.tucker_attn_decode(ctypes.byref(desc), x.data_ptr(), C.data_ptr(), U1.data_ptr(), U2.data_ptr(),
                                    U3.data_ptr(), Ct.data_ptr(), Ut1.data_ptr(), Ut2.data_ptr(), Ut3.data_ptr(),
                                    Kcache.data_ptr(), Vcache.data_ptr(), int(Lmax), cache_len.data_ptr(),
                                    int(bool(append)), out.data_ptr(), workspace.data_ptr(), workspace.numel(),
                                    _stream_ptr(dev))
    if rc != TA_OK:
        raise TuckerAttnError(rc, "tucker_attn_decode")
    return out


def tucker_attn_decode_static(x, C, U1, U2, U3, Ct, Ut1, Ut2, Ut3, Kcache, Vcache, cache_len, out, *, n_H: int,
                              rope: bool, rope_base: float = 10000.0, scale: float = 0.0, append: bool = True,
                              flags: int = 0):
    """Decode step for callers that cannot allocate: same arguments and result as
    tucker_attn_decode, but the output tensor `out` [B, d] is mandatory and no workspace is
    passed -- the library uses its built-in static scratch array (TA_STATIC_SCRATCH_BYTES).
    Neither this wrapper nor the C entry point allocates device memory.  Raises
    TuckerAttnError("workspace too small") when the problem needs more scratch than that.
    Calls share the one array: do not let two of them overlap on the GPU."""
    torch = _torch()
    lib = load_library()
    if x.dim() != 2:
        raise ValueError("x must be [B, d_model]")
    B, d = x.shape
    dev, dt = x.device, x.dtype
    _check(x, "x", (B, d), dt, dev)
    r, t = _weights_check((C, U1, U2, U3, Ct, Ut1, Ut2, Ut3), d, n_H, dt, dev)
    Lmax = Kcache.shape[1]
    _check(Kcache, "Kcache", (B, Lmax, r[2]), dt, dev)
    _check(Vcache, "Vcache", (B, Lmax, t[2]), dt, dev)
    _check(cache_len, "cache_len", (B,), torch.int32, dev)
    _check(out, "out", (B, d), dt, dev)
    desc = make_desc(B=B, N=1, d_model=d, n_H=n_H, r=r, t=t, causal=True, rope=rope, rope_base=rope_base,
                     pos0=0, scale=scale, dtype=_dtype_code(x), flags=flags)
    with torch.cuda.device(dev):
        rc = lib.tucker_attn_decode_static(ctypes.byref(desc), x.data_ptr(), C.data_ptr(), U1.data_ptr(),
                                           U2.data_ptr(), U3.data_ptr(), Ct.data_ptr(), Ut1.data_ptr(),
                                           Ut2.data_ptr(), Ut3.data_ptr(), Kcache.data_ptr(), Vcache.data_ptr(),
                                           int(Lmax), cache_len.data_ptr(), int(bool(append)), out.data_ptr(),
                                           _stream_ptr(dev))
    if rc != TA_OK:
        raise TuckerAttnError(rc, "tucker_attn_decode_static")
    return out


_PACK_KEYS = ("C", "U1", "U2", "U3", "Ct", "Ut1", "Ut2", "Ut3")


def _pack_outputs(shapes, like, out=None):
    torch = _torch()
    if out is None:
        return [torch.empty(sh, dtype=like.dtype, device=like.device) for sh in shapes]
    if len(out) != len(shapes):
        raise ValueError(f"out must hold {len(shapes)} tensors (C, U1, U2, U3, Ct, Ut1, Ut2, Ut3)")
    for name, t, sh in zip(_PACK_KEYS, out, shapes):
        _check(t, name, sh, like.dtype, like.device)
    return list(out)


def tucker_pack_gqa(WQ, WKg, WVg, WO, *, n_H: int, n_G: int, out=None):
    """GQA / MQA (n_G = n_H: MHA) weights as Tucker-attention weights; returns the list
    [C, U1, U2, U3, Ct, Ut1, Ut2, Ut3] of new device tensors (ranks (n_H, d, n_G d_H))."""
    torch = _torch()
    lib = load_library()
    d = WQ.shape[0]
    dev, dt = WQ.device, WQ.dtype
    if d % n_H or not (1 <= n_G <= n_H):
        raise ValueError("d_model must be a multiple of n_H and 1 <= n_G <= n_H")
    w = n_G * (d // n_H)
    _check(WQ, "WQ", (d, d), dt, dev)
    _check(WKg, "WKg", (d, w), dt, dev)
    _check(WVg, "WVg", (d, w), dt, dev)
    _check(WO, "WO", (d, d), dt, dev)
    outs = _pack_outputs([(n_H, d, w), (n_H, n_H), (d, d), (d, w), (n_H, d, w), (n_H, n_H), (d, d), (d, w)], WQ, out)
    with torch.cuda.device(dev):
        rc = lib.tucker_pack_gqa(int(d), int(n_H), int(n_G), _dtype_code(WQ), WQ.data_ptr(), WKg.data_ptr(),
                                 WVg.data_ptr(), WO.data_ptr(), *[o.data_ptr() for o in outs], _stream_ptr(dev))
    if rc != TA_OK:
        raise TuckerAttnError(rc, "tucker_pack_gqa")
    return outs


def tucker_pack_mha(WQ, WK, WV, WO, *, n_H: int, out=None):
    """MHA weights as Tucker-attention weights (ranks (n_H, d, d)); see tucker_pack_gqa."""
    torch = _torch()
    lib = load_library()
    d = WQ.shape[0]
    dev, dt = WQ.device, WQ.dtype
    if d % n_H:
        raise ValueError("d_model must be a multiple of n_H")
    for name, t in (("WQ", WQ), ("WK", WK), ("WV", WV), ("WO", WO)):
        _check(t, name, (d, d), dt, dev)
    outs = _pack_outputs([(n_H, d, d), (n_H, n_H), (d, d), (d, d), (n_H, d, d), (n_H, n_H), (d, d), (d, d)], WQ, out)
    with torch.cuda.device(dev):
        rc = lib.tucker_pack_mha(int(d), int(n_H), _dtype_code(WQ), WQ.data_ptr(), WK.data_ptr(), WV.data_ptr(),
                                 WO.data_ptr(), *[o.data_ptr() for o in outs], _stream_ptr(dev))
    if rc != TA_OK:
        raise TuckerAttnError(rc, "tucker_pack_mha")
    return outs


def tucker_pack_mla(WDQ, WUQ, WDKV, WUK, WDV, WUV, WO, *, n_H: int, out=None):
    """MLA (no RoPE) weights as Tucker-attention weights (ranks (n_H, dcq, dck) and
    (n_H, d, dck)); pass WDKV as WDV for a shared key / value latent."""
    torch = _torch()
    lib = load_library()
    d, dcq = WDQ.shape
    dck = WDKV.shape[1]
    dev, dt = WDQ.device, WDQ.dtype
    if d % n_H:
        raise ValueError("d_model must be a multiple of n_H")
    _check(WDQ, "WDQ", (d, dcq), dt, dev)
    _check(WUQ, "WUQ", (dcq, d), dt, dev)
    _check(WDKV, "WDKV", (d, dck), dt, dev)
    _check(WUK, "WUK", (dck, d), dt, dev)
    _check(WDV, "WDV", (d, dck), dt, dev)
    _check(WUV, "WUV", (dck, d), dt, dev)
    _check(WO, "WO", (d, d), dt, dev)
    outs = _pack_outputs([(n_H, dcq, dck), (n_H, n_H), (d, dcq), (d, dck), (n_H, d, dck), (n_H, n_H), (d, d), (d, dck)],
                         WDQ, out)
    with torch.cuda.device(dev):
        rc = lib.tucker_pack_mla(int(d), int(n_H), int(dcq), int(dck), _dtype_code(WDQ), WDQ.data_ptr(), WUQ.data_ptr(),
                                 WDKV.data_ptr(), WUK.data_ptr(), WDV.data_ptr(), WUV.data_ptr(), WO.data_ptr(),
                                 *[o.data_ptr() for o in outs], _stream_ptr(dev))
    if rc != TA_OK:
        raise TuckerAttnError(rc, "tucker_pack_mla")
    return outs


def tucker_mha_weight_tensors(WQ, WK, WV, WO, *, n_H: int):
    """The two n_H x d x d weight tensors of MHA weights (fp32): W[i] = WQ_i WK_i^T, Wt[i] = (WV_i WO_i)^T."""
    torch = _torch()
    d = WQ.shape[0]
    dev = WQ.device
    if d % n_H:
        raise ValueError("d_model must be a multiple of n_H")
    for name, t in (("WQ", WQ), ("WK", WK), ("WV", WV), ("WO", WO)):
        _check(t, name, (d, d), torch.float32, dev)
    W = torch.empty(n_H, d, d, dtype=torch.float32, device=dev)
    Wt = torch.empty_like(W)
    with torch.cuda.device(dev):
        rc = load_library().tucker_mha_weight_tensors(int(d), int(n_H), WQ.data_ptr(), WK.data_ptr(), WV.data_ptr(),
                                                      WO.data_ptr(), W.data_ptr(), Wt.data_ptr(), _stream_ptr(dev))
    if rc != TA_OK:
        raise TuckerAttnError(rc, "tucker_mha_weight_tensors")
    return W, Wt


def tucker_hosvd_init(W, ranks, *, workspace=None):
    """HOSVD of one weight tensor W [n_H, d, d] (fp32): returns (C [r1, r2, r3], U1 [n_H, r1], U2 [d, r2],
    U3 [d, r3], spectra), spectra = the singular values of the mode-1, mode-2 and mode-3 unfoldings
    ([n_H], [d], [d], each descending)."""
    torch = _torch()
    lib = load_library()
    if W.dim() != 3 or W.shape[1] != W.shape[2]:
        raise ValueError("W must be [n_H, d, d]")
    n_H, d, _ = W.shape
    dev = W.device
    _check(W, "W", (n_H, d, d), torch.float32, dev)
    r1, r2, r3 = (int(r) for r in ranks)
    f = dict(dtype=torch.float32, device=dev)
    C, U1 = torch.empty(r1, r2, r3, **f), torch.empty(n_H, r1, **f)
    U2, U3 = torch.empty(d, r2, **f), torch.empty(d, r3, **f)
    spectra = torch.empty(n_H + 2 * d, **f)
    need = int(lib.tucker_hosvd_workspace_bytes(int(d), int(n_H), r2, r3))
    if need == 0:
        raise ValueError("invalid sizes for tucker_hosvd_init")
    if workspace is None:
        workspace = alloc_workspace(need, dev)
    with torch.cuda.device(dev):
        rc = lib.tucker_hosvd_init(int(d), int(n_H), r1, r2, r3, W.data_ptr(), C.data_ptr(), U1.data_ptr(), U2.data_ptr(),
                                   U3.data_ptr(), spectra.data_ptr(), workspace.data_ptr(), workspace.numel(),
                                   _stream_ptr(dev))
    if rc != TA_OK:
        raise TuckerAttnError(rc, "tucker_hosvd_init")
    return C, U1, U2, U3, (spectra[:n_H], spectra[n_H:n_H + d], spectra[n_H + d:])


def probe_mma_rate(mode: int, N: int, iters: int = 256, n_blocks: int = 148) -> float:
    """Cycles per tcgen05.mma 128 x N x 16 for an operand source / layout (see tucker_probe_mma_rate): the
    slowest block's count divided by the number of MMAs."""
    torch = _torch()
    dev = torch.device("cuda", torch.cuda.current_device())
    cycles = torch.zeros(n_blocks, dtype=torch.int64, device=dev)
    rc = load_library().tucker_probe_mma_rate(int(mode), int(N), int(iters), int(n_blocks), cycles.data_ptr(),
                                              _stream_ptr(dev))
    if rc != TA_OK:
        raise TuckerAttnError(rc, "tucker_probe_mma_rate")
    torch.cuda.synchronize()
    return float(cycles.max().item()) / (iters * 8)


def probe_plane_mix(tiles: int, r1: int, n_blocks: int = 148):
    """Runs the plane-mixing probe (see tucker_probe_plane_mix); returns (median cycles per tile over the
    blocks, kernel milliseconds by CUDA events)."""
    torch = _torch()
    dev = torch.device("cuda", torch.cuda.current_device())
    u1 = torch.randn(2, r1, device=dev, dtype=torch.float32)
    cycles = torch.zeros(n_blocks, dtype=torch.int64, device=dev)
    sink = torch.zeros(n_blocks * 256, dtype=torch.float32, device=dev)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ms = 0.0
    for _ in range(2):      # the second run is the measured one
        e0.record()
        rc = load_library().tucker_probe_plane_mix(int(tiles), int(r1), int(n_blocks), u1.data_ptr(), cycles.data_ptr(),
                                                   sink.data_ptr(), _stream_ptr(dev))
        e1.record()
        if rc != TA_OK:
            raise TuckerAttnError(rc, "tucker_probe_plane_mix")
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
    return float(cycles.median().item()) / tiles, ms


def selftest_wait_timeout(budget_us: int = 2000, device=None):
    """Runs the library's bounded-wait self-test; returns the int32 tensor [first wait returned,
    second wait returned, second wait's duration / 1024 cycles] (read it after synchronising)."""
    torch = _torch()
    dev = torch.device("cuda", torch.cuda.current_device()) if device is None else device
    out = torch.full((3,), -1, dtype=torch.int32, device=dev)
    with torch.cuda.device(dev):
        rc = load_library().tucker_attn_selftest_wait_timeout(int(budget_us), out.data_ptr(), _stream_ptr(dev))
    if rc != TA_OK:
        raise TuckerAttnError(rc, "tucker_attn_selftest_wait_timeout")
    return out


def last_device_error(device=None) -> int:
    """Synchronises the current stream and returns-and-clears the device error word."""
    torch = _torch()
    dev = torch.device("cuda", torch.cuda.current_device()) if device is None else device
    with torch.cuda.device(dev):
        return int(load_library().tucker_attn_last_device_error(_stream_ptr(dev)))


def sync_status(device=None) -> int:
    """Synchronises the current stream and folds the device error word into a status code (and clears
    it): TA_OK, or TA_ERR_DEVICE_TIMEOUT (-5) / TA_ERR_INVALID_ARG (-1) / TA_ERR_CUDA (-4)."""
    torch = _torch()
    dev = torch.device("cuda", torch.cuda.current_device()) if device is None else device
    with torch.cuda.device(dev):
        return int(load_library().tucker_attn_sync_status(_stream_ptr(dev)))


def bounds_checked() -> bool:
    """True when the loaded library was built with -DTA_BOUNDS_CHECK."""
    return bool(load_library().tucker_attn_bounds_checked())


def last_path() -> int:
    return int(load_library().tucker_attn_last_path())


def last_launch_count() -> int:
    return int(load_library().tucker_attn_last_launch_count())


def set_profile_events(start=None, stop=None) -> None:
    """Registers two torch.cuda.Event(enable_timing=True) objects (already recorded once, so
    that their handles exist) to be recorded around the dominant kernel of later calls;
    call with no arguments to unregister."""
    lib = load_library()
    if start is None and stop is None:
        rc = lib.tucker_attn_set_profile_events(None, None)
    else:
        rc = lib.tucker_attn_set_profile_events(start.cuda_event, stop.cuda_event)
    if rc != TA_OK:
        raise TuckerAttnError(rc, "tucker_attn_set_profile_events")

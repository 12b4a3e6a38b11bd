"""ctypes binding of libsbnn.so.  Names mirror the C entry points (include/sbnn.h) without the sbnn_ prefix."""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
SBNN_RELU, SBNN_BF16_TC, SBNN_OUT_CM, SBNN_BF16_GATHER = 1, 2, 4, 8
_lib = None


class SbnnError(RuntimeError):
    def __init__(self, code, name, detail):
        super().__init__(f"{name}: {detail}")
        self.code, self.name, self.detail = code, name, detail


class _View(C.Structure):
    _fields_ = [("Cout", C.c_int), ("KH", C.c_int), ("KW", C.c_int), ("Cin", C.c_int), ("G", C.c_int),
                ("ngroups", C.c_int), ("nnz_units", C.c_int64), ("group_ptr", C.c_void_p), ("idx", C.c_void_p),
                ("val", C.c_void_p), ("bias", C.c_void_p), ("tap_mask", C.c_void_p), ("gi", C.c_int),
                ("block_idx", C.c_void_p)]


def lib_path() -> str:
    return os.path.join(_HERE, "libsbnn.so")


def lib():
    """Load libsbnn.so (built by paper_2310_19509_b200.build).  Fails loudly when it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    path = lib_path()
    if not os.path.exists(path):
        raise ImportError(f"{path} not found: build it with `python -m paper_2310_19509_b200.build`; "
                          "there is no fallback implementation")
    L = C.CDLL(path)
    P, I = C.c_void_p, C.c_int
    sig = {
        "sbnn_pack_weights": [P, P, P, I, I, I, I, I, P],
        "sbnn_pack_weights_pattern": [P, P, P, I, I, I, I, I, P],
        "sbnn_packed_get": [P, P],
        "sbnn_unpack_weights": [P, P, P],
        "sbnn_packed_free": [P],
        "sbnn_packed_save": [P, C.c_char_p],
        "sbnn_packed_load": [C.c_char_p, P],
        "sbnn_conv1x1_gs": [P, P, P, I, I, I, I, P],
        "sbnn_conv1x1_gs_tuned": [P, P, P, I, I, I, I, I, I, I, I, P],
        "sbnn_conv3x3_gs": [P, P, P, I, I, I, I, P],
        "sbnn_conv3x3_gs_cm": [P, P, I, P, I, I, I, I, I, P],
        "sbnn_conv1x1_gs_cm": [P, P, I, P, I, I, I, I, I, I, I, P],
        "sbnn_to_channel_major": [P, P, I, I, I, P],
        "sbnn_dwconv3x3": [P, P, P, P, I, I, I, I, I, I, P],
        "sbnn_dwconv3x3_cm": [P, P, P, I, P, I, I, I, I, I, I, I, P],
        "sbnn_dwconv3x3_conv1x1_gs_cm": [P, P, P, P, I, P, I, I, I, I, I, I, P],
        "sbnn_pack_dw_pattern": [P, P, I, I, P, P],
        "sbnn_dwconv3x3_pattern": [P, P, I, P, P, P, I, I, I, I, I, I, P],
        "sbnn_conv3x3_dense": [P, P, P, P, I, I, I, I, I, I, I, P],
        "sbnn_avgpool": [P, P, I, I, I, P],
        "sbnn_mobilenet_v1_create": [P, P, P, P, P, P, I, P],
        "sbnn_mobilenet_v1_forward": [P, P, P, I, P],
        "sbnn_mobilenet_v1_forward_prefix": [P, P, P, I, I, P],
        "sbnn_mobilenet_v1_run_layer": [P, I, P, P, I, P],
        "sbnn_mobilenet_v1_run_layer_cm": [P, I, P, P, I, P],
        "sbnn_mobilenet_v1_layer_shape": [I, P, P, P, P],
        "sbnn_mobilenet_v1_free": [P],
        "sbnn_get_async_status": [P],
        "sbnn_head_noalloc": [P, P, P, I, I, P],
        "sbnn_selftest_wait_timeout": [P],
        "sbnn_prepare": [P, I, I, I, I],
        "sbnn_selftest_fma_rate": [I, P, P],
        "sbnn_debug_set_packed_device": [P, I, P],
        "sbnn_debug_check_packed": [P, P],
        "sbnn_debug_poke_device_index": [P, C.c_longlong, I, P],
        "sbnn_debug_plan_conv3x3": [P, I, I, I, I, P, P, I, P, P, P],
    }
    for name, args in sig.items():
        f = getattr(L, name)
        f.argtypes, f.restype = args, I
    L.sbnn_status_str.argtypes, L.sbnn_status_str.restype = [I], C.c_char_p
    L.sbnn_last_error.argtypes, L.sbnn_last_error.restype = [], C.c_char_p
    _lib = L
    return L


def status_str(code: int) -> str:
    return lib().sbnn_status_str(code).decode()


def _check(code):
    if code != 0:
        L = lib()
        raise SbnnError(code, L.sbnn_status_str(code).decode(), L.sbnn_last_error().decode())


def _ptr(t):
    """Device pointer of a torch tensor (or a raw int / None)."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


class Packed:
    """Owner of an sbnn_packed handle."""

    def __init__(self, handle):
        self._h = handle

    @property
    def handle(self):
        return self._h

    def view(self):
        """Canonical arrays as numpy copies: dict(group_ptr, idx, val, bias, and the shape fields)."""
        v = _View()
        _check(lib().sbnn_packed_get(self._h, C.byref(v)))
        taps = v.KH * v.KW

        def arr(p, n, dt):
            if n == 0:
                return np.zeros(0, dtype=dt)
            return np.ctypeslib.as_array(C.cast(p, C.POINTER(C.c_byte * (n * np.dtype(dt).itemsize))).contents) \
                .view(dt).copy()

        return dict(Cout=v.Cout, KH=v.KH, KW=v.KW, Cin=v.Cin, G=v.G, ngroups=v.ngroups, nnz_units=v.nnz_units,
                    group_ptr=arr(v.group_ptr, v.ngroups + 1, np.int32), idx=arr(v.idx, v.nnz_units, np.int32),
                    val=arr(v.val, v.nnz_units * taps * v.G, np.float32).reshape(v.nnz_units, taps, v.G),
                    bias=arr(v.bias, v.Cout, np.float32),
                    tap_mask=arr(v.tap_mask, v.nnz_units, np.uint16) if v.tap_mask else None, gi=v.gi,
                    block_idx=arr(v.block_idx, v.nnz_units // 4, np.int32) if v.block_idx else None)

    def unpack(self):
        v = _View()
        _check(lib().sbnn_packed_get(self._h, C.byref(v)))
        w = np.empty((v.Cout, v.KH, v.KW, v.Cin), np.float32)
        m = np.empty((v.Cout, v.KH, v.KW, v.Cin), np.uint8)
        _check(lib().sbnn_unpack_weights(self._h, w.ctypes.data, m.ctypes.data))
        return w, m

    def save(self, path):
        """Write the layer to a packed-layer file (see sbnn_packed_save for the layout)."""
        _check(lib().sbnn_packed_save(self._h, os.fsencode(path)))

    def free(self):
        if self._h:
            lib().sbnn_packed_free(self._h)
            self._h = None

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass


def load_packed(path) -> Packed:
    """Read a packed-layer file written by Packed.save / sbnn_packed_save."""
    h = C.c_void_p()
    _check(lib().sbnn_packed_load(os.fsencode(path), C.byref(h)))
    return Packed(h)


def pack_weights(w, mask, bias, g, tap_patterns=False) -> Packed:
    """tap_patterns=True packs through sbnn_pack_weights_pattern (taps of a unit masked individually)."""
    w = np.ascontiguousarray(w, dtype=np.float32)
    mask = np.ascontiguousarray(mask, dtype=np.uint8)
    if w.ndim != 4 or mask.shape != w.shape:
        raise ValueError("w and mask must both be [Cout][KH][KW][Cin]")
    cout, kh, kw, cin = w.shape
    b = None if bias is None else np.ascontiguousarray(bias, dtype=np.float32)
    h = C.c_void_p()
    fn = lib().sbnn_pack_weights_pattern if tap_patterns else lib().sbnn_pack_weights
    _check(fn(w.ctypes.data, mask.ctypes.data, None if b is None else b.ctypes.data, cout, kh, kw, cin, int(g), C.byref(h)))
    return Packed(h)


def conv1x1_gs(w: Packed, x, y, n, h, wd, flags=SBNN_RELU, stream=None):
    _check(lib().sbnn_conv1x1_gs(w.handle, _ptr(x), _ptr(y), n, h, wd, flags, _stream(stream)))


def conv1x1_gs_tuned(w: Packed, x, y, n, h, wd, flags, p, gpw, nw, kc, stream=None):
    _check(lib().sbnn_conv1x1_gs_tuned(w.handle, _ptr(x), _ptr(y), n, h, wd, flags, p, gpw, nw, kc, _stream(stream)))


def conv1x1_gs_cm(w: Packed, xt, ldx, y, ldy, m, flags=SBNN_RELU, tile=(0, 0, 0, 0), stream=None):
    _check(lib().sbnn_conv1x1_gs_cm(w.handle, _ptr(xt), ldx, _ptr(y), ldy, m, flags, *tile, _stream(stream)))


def to_channel_major(x, xt, m, c, ld, stream=None):
    _check(lib().sbnn_to_channel_major(_ptr(x), _ptr(xt), m, c, ld, _stream(stream)))


def conv3x3_gs(w: Packed, x, y, n, h, wd, flags=SBNN_RELU, stream=None):
    _check(lib().sbnn_conv3x3_gs(w.handle, _ptr(x), _ptr(y), n, h, wd, flags, _stream(stream)))


def conv3x3_gs_cm(w: Packed, xt, ldx, y, ldy, n, h, wd, flags=SBNN_RELU, stream=None):
    _check(lib().sbnn_conv3x3_gs_cm(w.handle, _ptr(xt), ldx, _ptr(y), ldy, n, h, wd, flags, _stream(stream)))


def dwconv3x3(w, b, x, y, n, h, wd, c, stride, flags=SBNN_RELU, stream=None):
    _check(lib().sbnn_dwconv3x3(_ptr(w), _ptr(b), _ptr(x), _ptr(y), n, h, wd, c, stride, flags, _stream(stream)))


def dwconv3x3_cm(w, b, xt, ldx, yt, ldy, n, h, wd, c, stride, flags=SBNN_RELU, stream=None):
    _check(lib().sbnn_dwconv3x3_cm(_ptr(w), _ptr(b), _ptr(xt), ldx, _ptr(yt), ldy, n, h, wd, c, stride, flags, _stream(stream)))


def dwconv3x3_conv1x1_gs_cm(pw: Packed, dw_w, dw_b, xt, ldx, yt, ldy, n, h, wd, dw_flags=SBNN_RELU, pw_flags=SBNN_RELU, stream=None):
    """Depthwise 3x3 (stride 1) + group-sparse 1x1 as one kernel on channel-major tensors."""
    _check(lib().sbnn_dwconv3x3_conv1x1_gs_cm(pw.handle, _ptr(dw_w), _ptr(dw_b), _ptr(xt), ldx, _ptr(yt), ldy, n, h, wd,
                                              dw_flags, pw_flags, _stream(stream)))


def pack_dw_pattern(w, mask, go):
    """Host-side: dense depthwise weights [3][3][C] and a 3:9 pattern mask -> (pattern uint8 [C/go], w6 fp32 [3][2][C])."""
    w = np.ascontiguousarray(w, dtype=np.float32)
    mask = np.ascontiguousarray(mask, dtype=np.uint8)
    if w.ndim != 3 or w.shape[:2] != (3, 3) or mask.shape != w.shape:
        raise ValueError("w and mask must both be [3][3][C]")
    c = w.shape[2]
    pattern = np.zeros(max(c // max(int(go), 1), 1), dtype=np.uint8)
    w6 = np.zeros((3, 2, c), dtype=np.float32)
    _check(lib().sbnn_pack_dw_pattern(w.ctypes.data, mask.ctypes.data, c, int(go), pattern.ctypes.data, w6.ctypes.data))
    return pattern, w6


def dwconv3x3_pattern(w6, pattern, go, b, x, y, n, h, wd, c, stride, flags=SBNN_RELU, stream=None):
    _check(lib().sbnn_dwconv3x3_pattern(_ptr(w6), _ptr(pattern), int(go), _ptr(b), _ptr(x), _ptr(y), n, h, wd, c, stride,
                                        flags, _stream(stream)))


def conv3x3_dense(w, b, x, y, n, h, wd, cin, cout, stride, flags=SBNN_RELU, stream=None):
    _check(lib().sbnn_conv3x3_dense(_ptr(w), _ptr(b), _ptr(x), _ptr(y), n, h, wd, cin, cout, stride, flags,
                                    _stream(stream)))


def avgpool(x, y, n, hw, c, stream=None):
    _check(lib().sbnn_avgpool(_ptr(x), _ptr(y), n, hw, c, _stream(stream)))


def head_noalloc(fc: Packed, x, logits, n, hw, stream=None):
    """Average pool + classifier through the library's fixed scratch array; allocates nothing."""
    _check(lib().sbnn_head_noalloc(fc.handle, _ptr(x), _ptr(logits), n, hw, _stream(stream)))


def prepare(w: Packed, n, h, wd, flags=0):
    """Build ahead of time what compute calls of this layer would build on first use (see sbnn_prepare)."""
    _check(lib().sbnn_prepare(w.handle, n, h, wd, flags))


def selftest_fma_rate(iterations, stream=None) -> float:
    """Enqueue the register-only packed-FMA kernel; returns the flop it performs (time it with events)."""
    flop = C.c_double()
    _check(lib().sbnn_selftest_fma_rate(int(iterations), C.byref(flop), _stream(stream)))
    return flop.value


def debug_set_packed_device(w: Packed, device) -> int:
    """Test hook: overwrite the device recorded in a packed layer; returns the previous value."""
    prev = C.c_int()
    _check(lib().sbnn_debug_set_packed_device(w.handle, int(device), C.byref(prev)))
    return prev.value


def debug_check_packed(w: Packed, stream=None):
    """Enqueue the device-side consistency check of a packed layer (result through get_async_status)."""
    _check(lib().sbnn_debug_check_packed(w.handle, _stream(stream)))


def debug_plan_conv3x3(block_ptr, nrow, ncta):
    """Work plan of the pipelined 3x3 kernel for a block table [ntiles][nchunks + 1] (int32 numpy, host): returns
    (cta_ptr [ncta + 1], segs [nsegs][8] = bx, by, k0, k1, part, nparts, slot, counter, nslots, ncounters)."""
    bp = np.ascontiguousarray(block_ptr, dtype=np.int32)
    ntiles, nchunks = bp.shape[0], bp.shape[1] - 1
    cap = ntiles * nrow + 2 * ncta + 8
    cta_ptr = np.zeros(ncta + 1, dtype=np.int32)
    segs = np.zeros((cap, 8), dtype=np.int32)
    nsegs, nslots, ncounters = C.c_int(), C.c_int(), C.c_int()
    _check(lib().sbnn_debug_plan_conv3x3(bp.ctypes.data, ntiles, nchunks, int(nrow), int(ncta), cta_ptr.ctypes.data,
                                         segs.ctypes.data, cap, C.byref(nsegs), C.byref(nslots), C.byref(ncounters)))
    return cta_ptr, segs[:nsegs.value].copy(), nslots.value, ncounters.value


def debug_poke_device_index(w: Packed, unit, value) -> int:
    """Test hook: overwrite one index of the device copy; returns the previous value."""
    prev = C.c_int()
    _check(lib().sbnn_debug_poke_device_index(w.handle, int(unit), int(value), C.byref(prev)))
    return prev.value


def selftest_wait_timeout(stream=None):
    """Enqueue the diagnostic kernel whose bounded wait expires (see sbnn_selftest_wait_timeout)."""
    _check(lib().sbnn_selftest_wait_timeout(_stream(stream)))


def get_async_status(stream=None):
    _check(lib().sbnn_get_async_status(_stream(stream)))


def mobilenet_v1_layer_shape(layer):
    a, b, c, d = C.c_int(), C.c_int(), C.c_int(), C.c_int()
    _check(lib().sbnn_mobilenet_v1_layer_shape(layer, C.byref(a), C.byref(b), C.byref(c), C.byref(d)))
    return a.value, b.value, c.value, d.value


class MobileNetV1:
    """sbnn_mobilenet_v1_create / forward / run_layer / free.

    pw: 13 Packed pointwise layers; fc: Packed classifier; dw_w, dw_b: 13 device tensors each;
    conv0_w, conv0_b: device tensors.  The object keeps references so the memory outlives the handle.
    """

    def __init__(self, pw, fc, dw_w, dw_b, conv0_w, conv0_b, max_batch):
        assert len(pw) == 13 and len(dw_w) == 13 and len(dw_b) == 13
        self._keep = (list(pw), fc, list(dw_w), list(dw_b), conv0_w, conv0_b)
        PA = C.c_void_p * 13
        pws = PA(*[p.handle for p in pw])
        dws = PA(*[_ptr(t) for t in dw_w])
        dbs = PA(*[_ptr(t) for t in dw_b])
        h = C.c_void_p()
        _check(lib().sbnn_mobilenet_v1_create(pws, fc.handle, dws, dbs, _ptr(conv0_w), _ptr(conv0_b), max_batch,
                                              C.byref(h)))
        self._h = h

    def forward(self, x, logits, n, stream=None):
        _check(lib().sbnn_mobilenet_v1_forward(self._h, _ptr(x), _ptr(logits), n, _stream(stream)))

    def forward_prefix(self, x, out, n, last_layer, stream=None):
        """Layers 0..last_layer as forward launches them; the last one's output (chain layout) goes to `out`."""
        _check(lib().sbnn_mobilenet_v1_forward_prefix(self._h, _ptr(x), _ptr(out), n, int(last_layer), _stream(stream)))

    def run_layer(self, layer, x, y, n, stream=None):
        _check(lib().sbnn_mobilenet_v1_run_layer(self._h, layer, _ptr(x), _ptr(y), n, _stream(stream)))

    def run_layer_cm(self, layer, x, y, n, stream=None):
        """One layer on the chain's channel-major buffers (no layout conversion)."""
        _check(lib().sbnn_mobilenet_v1_run_layer_cm(self._h, layer, _ptr(x), _ptr(y), n, _stream(stream)))

    def free(self):
        if self._h:
            lib().sbnn_mobilenet_v1_free(self._h)
            self._h = None

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass

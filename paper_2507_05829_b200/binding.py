"""ctypes binding of include/lop.h.  Names and argument order follow the C header."""
import ctypes
import os
from ctypes import POINTER, Structure, byref, c_char_p, c_double, c_float, c_int, c_int32, c_size_t, c_uint, c_void_p

from . import build as _build

LIB_PATH = _build.LIB

LOP_F32, LOP_BF16 = 0, 1
LOP_CONV2D, LOP_MAXPOOL2D, LOP_LINEAR = 0, 1, 2
LOP_ACT_NONE, LOP_ACT_RELU, LOP_ACT_SILU = 0, 1, 2
LOP_RES_NONE, LOP_RES_PRE_ACT, LOP_RES_POST_ACT = 0, 1, 2
LOP_INPUT, LOP_NO_RESIDUAL = -1, -2
LOP_FLAG_REUSE_HALO, LOP_FLAG_TIME_LAYERS, LOP_FLAG_FORCE_SIMT, LOP_FLAG_PER_LAYER, LOP_FLAG_COPY_ENGINE, LOP_FLAG_DEBUG_BOUNDS = 1, 2, 4, 8, 16, 32

# every symbol include/lop.h declares
EXPORTS = [
    "lop_plan", "lop_plan_destroy", "lop_plan_num_bands", "lop_plan_num_layers", "lop_plan_get_range",
    "lop_plan_out_shape", "lop_plan_set_params", "lop_plan_workspace_bytes", "lop_plan_staging_bytes",
    "lop_plan_flops", "lop_run_whole", "lop_run_band", "lop_run_layer", "lop_run_banded", "lop_copy_band", "lop_fetch_band", "lop_run_pipelined",
    "lop_plan_last_timing", "lop_plan_layer_time", "lop_plan_layer_kernel", "lop_plan_last_launches", "lop_plan_last_copies",
    "lop_plan_check_device", "lop_plan_set_wait_limit", "lop_run_pipelined_withheld", "lop_plan_layer_offset", "lop_plan_layer_stored", "lop_run_whole_static", "lop_run_chain_banded", "lop_run_chain_pipelined", "lop_plan_shard", "lop_run_shard",
    "lop_strerror", "lop_last_error",
]
LOP_STATIC_SCRATCH_BYTES = 16 << 20


class LopError(RuntimeError):
    def __init__(self, status, message):
        super().__init__("lop status %d: %s" % (status, message))
        self.status = status


class LopLayer(Structure):
    _fields_ = [(n, c_int32) for n in ("op", "cin", "cout", "kh", "kw", "sh", "sw", "ph", "pw", "dh", "dw", "act",
                                        "input_from", "residual_from", "residual_pos", "reserved")] + \
               [("weight", c_void_p), ("scale", c_void_p), ("shift", c_void_p)]


class LopRange(Structure):
    _fields_ = [(n, c_int32) for n in ("out_lo", "out_hi", "in_lo", "in_hi", "pad_top", "pad_bot", "new_lo", "reserved")]

    def astuple(self):
        return (self.out_lo, self.out_hi, self.in_lo, self.in_hi, self.pad_top, self.pad_bot, self.new_lo)


class LopTiming(Structure):
    _fields_ = [("total_ms", c_float), ("copy_ms", c_float), ("first_copy_ms", c_float), ("n_copies", c_int32),
                ("reserved", c_int32)]


_lib = None


def lib():
    """The loaded C-ABI library.  Builds it in-tree when missing; raises if that is impossible."""
    global _lib
    if _lib is not None:
        return _lib
    path = LIB_PATH
    if _build.needs_build():
        try:
            path = _build.build()
        except Exception as e:  # no silent fallback: there is no other implementation
            if not os.path.exists(LIB_PATH):
                raise ImportError("liblop_b200.so is missing and could not be built: %s" % e)
    L = ctypes.CDLL(path)
    L.lop_plan.argtypes = [POINTER(LopLayer), c_int, c_int, c_int, c_int, c_int, c_int, c_int, c_uint, POINTER(c_void_p)]
    L.lop_plan_destroy.argtypes = [c_void_p]
    L.lop_plan_destroy.restype = None
    L.lop_plan_num_bands.argtypes = [c_void_p]
    L.lop_plan_num_layers.argtypes = [c_void_p]
    L.lop_plan_get_range.argtypes = [c_void_p, c_int, c_int, POINTER(LopRange)]
    L.lop_plan_out_shape.argtypes = [c_void_p, c_int, POINTER(c_int), POINTER(c_int), POINTER(c_int)]
    L.lop_plan_set_params.argtypes = [c_void_p, c_int, c_void_p, c_void_p, c_void_p]
    L.lop_plan_workspace_bytes.argtypes = [c_void_p]
    L.lop_plan_workspace_bytes.restype = c_size_t
    L.lop_plan_staging_bytes.argtypes = [c_void_p]
    L.lop_plan_staging_bytes.restype = c_size_t
    L.lop_plan_flops.argtypes = [c_void_p]
    L.lop_plan_flops.restype = c_double
    L.lop_run_whole.argtypes = [c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]
    L.lop_run_band.argtypes = [c_void_p, c_int, c_void_p, c_void_p, c_void_p, c_void_p]
    L.lop_run_layer.argtypes = [c_void_p, c_int, c_int, c_int, c_void_p, c_void_p, c_void_p, c_void_p]
    L.lop_run_banded.argtypes = [c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]
    L.lop_copy_band.argtypes = [c_void_p, c_int, c_void_p, c_void_p, c_void_p]
    L.lop_fetch_band.argtypes = [c_void_p, c_int, c_void_p, c_void_p, c_void_p, c_void_p]
    L.lop_run_pipelined.argtypes = [c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]
    L.lop_plan_last_timing.argtypes = [c_void_p, POINTER(LopTiming)]
    L.lop_plan_layer_time.argtypes = [c_void_p, c_int, c_int, POINTER(c_float)]
    L.lop_plan_layer_kernel.argtypes = [c_void_p, c_int]
    L.lop_plan_layer_offset.argtypes = [c_void_p, c_int, POINTER(c_size_t)]
    L.lop_plan_layer_stored.argtypes = [c_void_p, c_int]
    L.lop_plan_last_launches.argtypes = [c_void_p]
    L.lop_plan_last_copies.argtypes = [c_void_p]
    L.lop_plan_check_device.argtypes = [c_void_p, c_void_p]
    L.lop_plan_set_wait_limit.argtypes = [c_void_p, c_uint]
    L.lop_run_pipelined_withheld.argtypes = [c_void_p, c_int, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]
    L.lop_run_whole_static.argtypes = [c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]
    L.lop_run_chain_banded.argtypes = [POINTER(c_void_p), c_int, c_void_p, POINTER(c_void_p), POINTER(c_void_p), c_void_p]
    L.lop_run_chain_pipelined.argtypes = [POINTER(c_void_p), c_int, c_void_p, c_void_p, POINTER(c_void_p), POINTER(c_void_p), c_void_p]
    L.lop_plan_shard.argtypes = [c_void_p, c_int, c_int] + [POINTER(c_int)] * 6
    L.lop_run_shard.argtypes = [c_void_p, c_int, c_int, c_void_p, c_void_p, c_void_p, c_void_p]
    L.lop_strerror.argtypes = [c_int]
    L.lop_strerror.restype = c_char_p
    L.lop_last_error.restype = c_char_p
    _lib = L
    return L


def _check(rc):
    if rc < 0:
        raise LopError(rc, lib().lop_last_error().decode() or lib().lop_strerror(rc).decode())
    return rc


def make_layer_array(layers):
    """``layers``: objects with the fields of lop_layer (weight/scale/shift: device addresses or None)."""
    arr = (LopLayer * len(layers))()
    for a, l in zip(arr, layers):
        for n in ("op", "cin", "cout", "kh", "kw", "sh", "sw", "ph", "pw", "dh", "dw", "act", "input_from",
                  "residual_from", "residual_pos"):
            setattr(a, n, int(getattr(l, n)))
        a.weight = getattr(l, "weight_ptr", None)
        a.scale = getattr(l, "scale_ptr", None)
        a.shift = getattr(l, "shift_ptr", None)
    return arr


def _ptr_array(values):
    return (c_void_p * len(values))(*values)


def run_chain_banded(plans, in_dev, outs_dev, workspaces, stream):
    """lop_run_chain_banded: ``plans`` are :class:`Plan` objects, the rest device addresses."""
    _check(lib().lop_run_chain_banded(_ptr_array([p._h.value for p in plans]), len(plans), in_dev, _ptr_array(outs_dev),
                                      _ptr_array(workspaces), stream))


def run_chain_pipelined(plans, in_host, staging_dev, outs_dev, workspaces, stream):
    """lop_run_chain_pipelined."""
    _check(lib().lop_run_chain_pipelined(_ptr_array([p._h.value for p in plans]), len(plans), in_host, staging_dev,
                                         _ptr_array(outs_dev), _ptr_array(workspaces), stream))


class Plan:
    """Owns a lop_plan_t*; every method is the C function of the same name minus the ``lop_`` prefix."""

    def __init__(self, layers, N, H, W, C, dtype, n_bands, flags=0):
        self._h = c_void_p()
        self.n_layers = len(layers)
        arr = make_layer_array(layers) if layers else None
        _check(lib().lop_plan(arr, len(layers), N, H, W, C, dtype, n_bands, flags, byref(self._h)))

    def destroy(self):
        if self._h:
            lib().lop_plan_destroy(self._h)
            self._h = c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    def num_bands(self):
        return _check(lib().lop_plan_num_bands(self._h))

    def num_layers(self):
        return _check(lib().lop_plan_num_layers(self._h))

    def get_range(self, band, layer):
        r = LopRange()
        _check(lib().lop_plan_get_range(self._h, band, layer, byref(r)))
        return r

    def out_shape(self, layer):
        h, w, c = c_int(), c_int(), c_int()
        _check(lib().lop_plan_out_shape(self._h, layer, byref(h), byref(w), byref(c)))
        return h.value, w.value, c.value

    def set_params(self, layer, weight, scale, shift):
        _check(lib().lop_plan_set_params(self._h, layer, weight, scale, shift))

    def workspace_bytes(self):
        return lib().lop_plan_workspace_bytes(self._h)

    def staging_bytes(self):
        return lib().lop_plan_staging_bytes(self._h)

    def flops(self):
        return lib().lop_plan_flops(self._h)

    def run_whole(self, in_dev, out_dev, ws, stream):
        _check(lib().lop_run_whole(self._h, in_dev, out_dev, ws, stream))

    def run_band(self, band, in_dev, out_dev, ws, stream):
        _check(lib().lop_run_band(self._h, band, in_dev, out_dev, ws, stream))

    def run_layer(self, layer, row_lo, row_hi, in_dev, out_dev, ws, stream):
        _check(lib().lop_run_layer(self._h, layer, row_lo, row_hi, in_dev, out_dev, ws, stream))

    def run_banded(self, in_dev, out_dev, ws, stream):
        _check(lib().lop_run_banded(self._h, in_dev, out_dev, ws, stream))

    def copy_band(self, band, in_host, staging_dev, stream):
        _check(lib().lop_copy_band(self._h, band, in_host, staging_dev, stream))

    def fetch_band(self, band, in_host, staging_dev, ws, stream):
        """lop_fetch_band: band == -1 brings every band's rows."""
        _check(lib().lop_fetch_band(self._h, band, in_host, staging_dev, ws, stream))

    def shard(self, rank, world):
        """(band_lo, band_hi, row_lo, row_hi, in_lo, in_hi) of device ``rank`` of ``world`` (host only)."""
        v = [c_int(0) for _ in range(6)]
        _check(lib().lop_plan_shard(self._h, rank, world, *[byref(x) for x in v]))
        return tuple(x.value for x in v)

    def run_shard(self, band_lo, band_hi, in_dev, out_dev, ws, stream):
        _check(lib().lop_run_shard(self._h, band_lo, band_hi, in_dev, out_dev, ws, stream))

    def run_pipelined(self, in_host, staging_dev, out_dev, ws, stream):
        _check(lib().lop_run_pipelined(self._h, in_host, staging_dev, out_dev, ws, stream))

    def last_timing(self):
        t = LopTiming()
        _check(lib().lop_plan_last_timing(self._h, byref(t)))
        return t

    def layer_time(self, band, layer):
        ms = c_float()
        _check(lib().lop_plan_layer_time(self._h, band, layer, byref(ms)))
        return ms.value

    def layer_kernel(self, layer):
        return _check(lib().lop_plan_layer_kernel(self._h, layer))

    def layer_offset(self, layer):
        off = c_size_t()
        _check(lib().lop_plan_layer_offset(self._h, layer, byref(off)))
        return off.value

    def layer_stored(self, layer):
        return bool(_check(lib().lop_plan_layer_stored(self._h, layer)))

    def last_launches(self):
        return _check(lib().lop_plan_last_launches(self._h))

    def last_copies(self):
        return _check(lib().lop_plan_last_copies(self._h))

    def run_whole_static(self, in_dev, out_dev, status_dev, stream):
        """lop_run_whole_static: no workspace argument, nothing is allocated (see include/lop.h)."""
        _check(lib().lop_run_whole_static(self._h, in_dev, out_dev, status_dev, stream))

    def set_wait_limit(self, polls):
        _check(lib().lop_plan_set_wait_limit(self._h, polls))

    def run_pipelined_withheld(self, band, in_host, staging_dev, out_dev, ws, stream):
        _check(lib().lop_run_pipelined_withheld(self._h, band, in_host, staging_dev, out_dev, ws, stream))

    def check_device(self, ws):
        _check(lib().lop_plan_check_device(self._h, ws))

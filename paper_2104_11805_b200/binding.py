"""ctypes binding of libsdnn.so: argument marshalling only, one Python method per C entry point.

Every step of the path runs inside the library's CUDA kernels.  There is no fallback: if the
library is missing or no CUDA device is present, calls raise.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsdnn.so")

FLAG_BWD_ATOMICS, FLAG_BWD_CSC, FLAG_KEEP_DEBUG, FLAG_SKIP_DEAD, FLAG_NO_GRAPH, FLAG_NO_PDL = 0x01, 0x02, 0x04, 0x08, 0x10, 0x20
FLAG_BWD_ONE_LAUNCH = 0x80
FLAG_ONE_TILE = 0x40
FLAG_REORDER = 0x100
FLAG_SMEM_WINDOWS = 0x200
FLAG_IDX32 = 0x400
ACT_CLAMPED_RELU, ACT_SIGMOID = 0, 1

STATUS = {0: "SDNN_OK", -1: "SDNN_ERR_INVALID_ARG", -2: "SDNN_ERR_BAD_CSR", -3: "SDNN_ERR_OOM", -4: "SDNN_ERR_CUDA",
          -5: "SDNN_ERR_STATE", -6: "SDNN_ERR_UNIMPLEMENTED"}


class SdnnConfig(ctypes.Structure):
    _fields_ = [("activation", ctypes.c_int32), ("clamp", ctypes.c_float), ("max_batch", ctypes.c_int32),
                ("train", ctypes.c_int32), ("update_bias", ctypes.c_int32), ("flags", ctypes.c_uint32),
                ("cuda_stream", ctypes.c_void_p), ("device", ctypes.c_int32)]


class SdnnError(RuntimeError):
    def __init__(self, code: int, message: str):
        super().__init__(f"{STATUS.get(code, code)}: {message}")
        self.code = code
        self.message = message


_vp, _i32, _i64, _f32 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_float
_PROTOS = {
    "sdnn_create": (ctypes.c_int, [ctypes.POINTER(_vp), _i32, _i32, _vp, _vp, _vp, _vp, ctypes.POINTER(SdnnConfig)]),
    "sdnn_create_deferred": (ctypes.c_int, [ctypes.POINTER(_vp), _i32, _i32, _vp, ctypes.POINTER(SdnnConfig)]),
    "sdnn_load_layer": (ctypes.c_int, [_vp, _i32, _vp, _vp, _vp, _vp]),
    "sdnn_finalize": (ctypes.c_int, [_vp]),
    "sdnn_infer_batch": (ctypes.c_int, [_vp, _vp, _i64, _vp, _vp, _vp, _i64, ctypes.POINTER(_i64)]),
    "sdnn_infer_batch_host": (ctypes.c_int, [_vp, _vp, _i64, _vp, _vp, _vp, _i64, ctypes.POINTER(_i64)]),
    "sdnn_train_step": (ctypes.c_int, [_vp, _vp, _vp, _i32, _f32, ctypes.POINTER(_f32)]),
    "sdnn_train_step_host": (ctypes.c_int, [_vp, _vp, _vp, _i32, _f32, ctypes.POINTER(_f32)]),
    "sdnn_train_step_averaged": (ctypes.c_int, [_vp, _vp, _vp, _i32, _f32, ctypes.POINTER(_f32)]),
    "sdnn_get_weights": (ctypes.c_int, [_vp, _i32, _vp, _vp]),
    "sdnn_set_weights": (ctypes.c_int, [_vp, _i32, _vp, _vp]),
    "sdnn_get_activations": (ctypes.c_int, [_vp, _i32, _vp]),
    "sdnn_get_delta": (ctypes.c_int, [_vp, _i32, _vp]),
    "sdnn_get_gradient": (ctypes.c_int, [_vp, _i32, _vp]),
    "sdnn_mirror_mismatches": (ctypes.c_int, [_vp, _i32, ctypes.POINTER(_i64)]),
    "sdnn_probe_gather_rate": (ctypes.c_int, [_i32, _i64, ctypes.POINTER(ctypes.c_double)]),
    "sdnn_probe_gather_inflight": (ctypes.c_int, [_i64, _i32, _i32, ctypes.POINTER(ctypes.c_double)]),
    "sdnn_probe_layer_boundary": (ctypes.c_int, [_i32, _i32, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double)]),
    "sdnn_probe_tma_gather_rate": (ctypes.c_int, [_i32, _i64, _i32, ctypes.POINTER(ctypes.c_double)]),
    "sdnn_probe_mixed_gather": (ctypes.c_int, [_i32, _i64, _i32, _i32, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double)]),
    "sdnn_probe_word_rate": (ctypes.c_int, [_i32, _i64, ctypes.POINTER(ctypes.c_double)]),
    "sdnn_probe_smem_gather_rate": (ctypes.c_int, [_i32, _i32, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(_i32)]),
    "sdnn_get_phase_times": (ctypes.c_int, [_vp, ctypes.POINTER(_f32), ctypes.POINTER(_f32)]),
    "sdnn_get_liveness": (ctypes.c_int, [_vp, _vp]),
    "sdnn_infer_noalloc": (ctypes.c_int, [_i32, _i32, _vp, _vp, _vp, _vp, _vp, _vp, _i32, _vp, _f32, _vp]),
    "sdnn_windowed_layers": (_i32, [_vp]),
    "sdnn_grouped_layers": (_i32, [_vp]),
    "sdnn_cluster_layer": (ctypes.c_int, [_i32, _vp, _vp, _i32, _i32, _vp, _vp, ctypes.POINTER(_i32), ctypes.POINTER(_i32)]),
    "sdnn_infer_noalloc_bad_columns": (ctypes.c_int, [ctypes.POINTER(_i64)]),
    "sdnn_kernel_launches": (_i64, [_vp]),
    "sdnn_infer_tile_width": (_i32, [_vp]),
    "sdnn_infer_tiles_in_flight": (_i32, [_vp]),
    "sdnn_device_bytes": (_i64, [_vp]),
    "sdnn_destroy": (None, [_vp]),
    "sdnn_last_error": (ctypes.c_char_p, [_vp]),
    "sdnn_version": (ctypes.c_char_p, []),
}

_lib = None


def exported_symbols():
    """Names the header declares (and the library must export)."""
    return sorted(_PROTOS)


def load_library(path: str | None = None):
    """dlopen libsdnn.so and attach prototypes.  Raises if the library has not been built."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or LIB_PATH
    if not os.path.exists(p):
        raise SdnnError(-4, f"{p} not found: build it first (python -m paper_2104_11805_b200.build); "
                            "there is no CPU fallback")
    lib = ctypes.CDLL(p)
    for name, (res, args) in _PROTOS.items():
        fn = getattr(lib, name)          # AttributeError if a declared symbol is not exported
        fn.restype, fn.argtypes = res, args
    if path is None:
        _lib = lib
    return lib


def _np(a, dtype):
    return np.ascontiguousarray(a, dtype=dtype)


def _addr(x):
    """Device or host address of a torch tensor / numpy array / int / None."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if isinstance(x, np.ndarray):
        return x.ctypes.data
    return x.data_ptr()      # torch tensor


NOALLOC_MAX_TILE_FLOATS = 1 << 20


def infer_noalloc(n_layers, n_neurons, row_ptr, col_idx, values, layer_offset, bias, x0, n_inputs, y_out,
                  clamp=32.0, stream=None):
    """sdnn_infer_noalloc: forward through the whole net with no handle and no allocation.

    For callers that may not allocate device memory at call time (the device is fully reserved by
    another allocator, an allocation's implicit synchronisation is not acceptable, or their interface
    forbids it): the net and the inputs/outputs are the caller's device arrays (anything with
    data_ptr(), or raw addresses), the activation scratch is a fixed array inside the library.
    layer_offset is a host sequence of element offsets (multiples of 4).  Raises SdnnError if
    n_neurons * padded(n_inputs) exceeds NOALLOC_MAX_TILE_FLOATS.  Calls sharing the scratch must not
    overlap on the GPU."""
    lib = load_library()
    off = _np(layer_offset, np.int64)
    rc = lib.sdnn_infer_noalloc(n_layers, n_neurons, _addr(row_ptr), _addr(col_idx), _addr(values), off.ctypes.data,
                                _addr(bias), _addr(x0), n_inputs, _addr(y_out), clamp, stream)
    if rc != 0:
        raise SdnnError(rc, (lib.sdnn_last_error(None) or b"").decode())


def infer_noalloc_bad_columns():
    """sdnn_infer_noalloc_bad_columns: out-of-range column indices that infer_noalloc met (and skipped) on this device."""
    lib = load_library()
    out = _i64(0)
    rc = lib.sdnn_infer_noalloc_bad_columns(ctypes.byref(out))
    if rc != 0:
        raise SdnnError(rc, (lib.sdnn_last_error(None) or b"").decode())
    return out.value


def probe_gather_rate(row_bytes, table_rows):
    """sdnn_probe_gather_rate: random rows of `row_bytes` bytes per second gathered out of a table of `table_rows` rows."""
    lib = load_library()
    out = ctypes.c_double(0.0)
    rc = lib.sdnn_probe_gather_rate(row_bytes, table_rows, ctypes.byref(out))
    if rc != 0:
        raise SdnnError(rc, (lib.sdnn_last_error(None) or b"").decode())
    return out.value


def probe_gather_inflight(table_rows, threads_per_sm, loads_in_flight):
    """sdnn_probe_gather_inflight: 64-byte random rows per second with exactly threads_per_sm / 2 * loads_in_flight rows
    in flight per SM."""
    lib = load_library()
    out = ctypes.c_double(0.0)
    rc = lib.sdnn_probe_gather_inflight(table_rows, threads_per_sm, loads_in_flight, ctypes.byref(out))
    if rc != 0:
        raise SdnnError(rc, (lib.sdnn_last_error(None) or b"").decode())
    return out.value


def probe_layer_boundary(ctas_per_sm, threads):
    """sdnn_probe_layer_boundary: (microseconds per grid-wide barrier inside one cooperative launch, microseconds per
    dependent launch of a graph-captured chain) for grids of ctas_per_sm CTAs of `threads` threads per SM."""
    lib = load_library()
    bar, lau = ctypes.c_double(0.0), ctypes.c_double(0.0)
    rc = lib.sdnn_probe_layer_boundary(ctas_per_sm, threads, ctypes.byref(bar), ctypes.byref(lau))
    if rc != 0:
        raise SdnnError(rc, (lib.sdnn_last_error(None) or b"").decode())
    return bar.value, lau.value


def cluster_layer(row_ptr, col_idx, col_cap=1536, row_cap=2048):
    """sdnn_cluster_layer: (group_of_row, col_label, n_groups, max_window) of one CSR pattern; n_groups == 0 and None
    arrays when the pattern has no block structure.  Host only."""
    lib = load_library()
    rp, ci = _np(row_ptr, np.int32), _np(col_idx, np.int32)
    n = len(rp) - 1
    grp, lab = np.empty(n, dtype=np.int32), np.empty(n, dtype=np.int32)
    ng, mw = ctypes.c_int32(0), ctypes.c_int32(0)
    rc = lib.sdnn_cluster_layer(n, rp.ctypes.data, ci.ctypes.data, col_cap, row_cap, grp.ctypes.data, lab.ctypes.data,
                                ctypes.byref(ng), ctypes.byref(mw))
    if rc != 0:
        raise SdnnError(rc, (lib.sdnn_last_error(None) or b"").decode())
    if ng.value == 0:
        return None, None, 0, 0
    return grp, lab, ng.value, mw.value


def probe_tma_gather_rate(row_bytes, table_rows, gather4):
    """sdnn_probe_tma_gather_rate: random rows per second fetched by the copy engine into shared memory (bulk copies
    per row, or four rows per tile::gather4 instruction)."""
    lib = load_library()
    out = ctypes.c_double(0.0)
    rc = lib.sdnn_probe_tma_gather_rate(row_bytes, table_rows, int(bool(gather4)), ctypes.byref(out))
    if rc != 0:
        raise SdnnError(rc, (lib.sdnn_last_error(None) or b"").decode())
    return out.value


def probe_mixed_gather(row_bytes, table_rows, tma_rounds, lsu_per_group):
    """sdnn_probe_mixed_gather: (seconds per launch, rows per launch) with the copy engine and the load instructions
    gathering side by side (either part may be 0)."""
    lib = load_library()
    sec, rows = ctypes.c_double(0.0), ctypes.c_double(0.0)
    rc = lib.sdnn_probe_mixed_gather(row_bytes, table_rows, tma_rounds, lsu_per_group, ctypes.byref(sec), ctypes.byref(rows))
    if rc != 0:
        raise SdnnError(rc, (lib.sdnn_last_error(None) or b"").decode())
    return sec.value, rows.value


def probe_word_rate(store, table_words):
    """sdnn_probe_word_rate: scattered 4-byte loads (store=False) or stores (store=True) per second."""
    lib = load_library()
    out = ctypes.c_double(0.0)
    rc = lib.sdnn_probe_word_rate(int(bool(store)), table_words, ctypes.byref(out))
    if rc != 0:
        raise SdnnError(rc, (lib.sdnn_last_error(None) or b"").decode())
    return out.value


def probe_smem_gather_rate(row_bytes, cluster_size):
    """sdnn_probe_smem_gather_rate: (rows per second, CTAs taking part) for random rows out of shared memory
    (cluster_size 1) or out of a cluster's distributed shared memory."""
    lib = load_library()
    out, ctas = ctypes.c_double(0.0), ctypes.c_int32(0)
    rc = lib.sdnn_probe_smem_gather_rate(row_bytes, cluster_size, ctypes.byref(out), ctypes.byref(ctas))
    if rc != 0:
        raise SdnnError(rc, (lib.sdnn_last_error(None) or b"").decode())
    return out.value, ctas.value


class Sdnn:
    """Owns one sdnn_t handle.  Method names mirror the C entry points (sdnn_ prefix dropped)."""

    def __init__(self, handle, n_layers, n_neurons, nnz, lib):
        self._h, self.n_layers, self.n_neurons, self.nnz, self._lib = handle, n_layers, n_neurons, list(nnz), lib

    # ---- construction -----------------------------------------------------------------------
    @staticmethod
    def _config(max_batch, train, clamp, update_bias, flags, stream, device, activation=0):
        return SdnnConfig(activation, clamp, max_batch, int(train), int(update_bias), flags, stream, device)

    @classmethod
    def create(cls, row_ptr, col_idx, values, bias, *, max_batch, train=False, clamp=32.0, update_bias=False,
               flags=0, stream=None, device=-1, activation=0):
        lib = load_library()
        L = len(col_idx)
        n = len(bias[0]) if L else 0
        rp = [_np(a, np.int32) for a in row_ptr]
        ci = [_np(a, np.int32) for a in col_idx]
        va = [_np(a, np.float32) for a in values]
        bi = [_np(a, np.float32) for a in bias]
        arr = lambda xs: (ctypes.c_void_p * max(L, 1))(*[x.ctypes.data for x in xs])
        cfg = cls._config(max_batch, train, clamp, update_bias, flags, stream, device, activation)
        h = ctypes.c_void_p()
        rc = lib.sdnn_create(ctypes.byref(h), L, n, arr(rp), arr(ci), arr(va), arr(bi), ctypes.byref(cfg))
        if rc != 0:
            raise SdnnError(rc, (lib.sdnn_last_error(None) or b"").decode())
        return cls(h, L, n, [len(c) for c in ci], lib)

    @classmethod
    def create_deferred(cls, n_layers, n_neurons, nnz_per_layer, *, max_batch, train=False, clamp=32.0,
                        update_bias=False, flags=0, stream=None, device=-1, activation=0):
        lib = load_library()
        nnz = _np(nnz_per_layer, np.int64)
        cfg = cls._config(max_batch, train, clamp, update_bias, flags, stream, device, activation)
        h = ctypes.c_void_p()
        rc = lib.sdnn_create_deferred(ctypes.byref(h), n_layers, n_neurons, nnz.ctypes.data, ctypes.byref(cfg))
        if rc != 0:
            raise SdnnError(rc, (lib.sdnn_last_error(None) or b"").decode())
        return cls(h, n_layers, n_neurons, nnz.tolist(), lib)

    def _check(self, rc):
        if rc != 0:
            raise SdnnError(rc, (self._lib.sdnn_last_error(self._h) or b"").decode())

    def load_layer(self, layer, row_ptr, col_idx, values, bias):
        rp, ci, va, bi = _np(row_ptr, np.int32), _np(col_idx, np.int32), _np(values, np.float32), _np(bias, np.float32)
        self._check(self._lib.sdnn_load_layer(self._h, layer, rp.ctypes.data, ci.ctypes.data, va.ctypes.data, bi.ctypes.data))

    def finalize(self):
        self._check(self._lib.sdnn_finalize(self._h))

    # ---- hot path ---------------------------------------------------------------------------
    def infer_batch(self, x0, n_inputs, y_out=None, nz_count_out=None, nz_index_out=None, nz_index_capacity=0,
                    want_total=False, host=False):
        """Device pointers (torch CUDA tensors) unless host=True (numpy / pinned torch CPU tensors).
        Returns the total id count when want_total (forces a stream sync), else None."""
        total = ctypes.c_int64(0)
        fn = self._lib.sdnn_infer_batch_host if host else self._lib.sdnn_infer_batch
        rc = fn(self._h, _addr(x0), n_inputs, _addr(y_out), _addr(nz_count_out), _addr(nz_index_out),
                nz_index_capacity, ctypes.byref(total) if want_total else None)
        self.last_total = total.value
        self._check(rc)
        return total.value if want_total else None

    def train_step(self, x0, target, B, eta, want_loss=False, host=False, averaged=False):
        """One minibatch step.  averaged=True: the averaged form (one backpropagated vector; device pointers only)."""
        loss = ctypes.c_float(0.0)
        if averaged and host:
            raise ValueError("the averaged step takes device pointers")
        fn = (self._lib.sdnn_train_step_averaged if averaged else
              self._lib.sdnn_train_step_host if host else self._lib.sdnn_train_step)
        self._check(fn(self._h, _addr(x0), _addr(target), B, eta, ctypes.byref(loss) if want_loss else None))
        return loss.value if want_loss else None

    # ---- state / inspection -----------------------------------------------------------------
    def get_weights(self, layer, want_bias=True):
        v = np.empty(self.nnz[layer], dtype=np.float32)
        b = np.empty(self.n_neurons, dtype=np.float32) if want_bias else None
        self._check(self._lib.sdnn_get_weights(self._h, layer, v.ctypes.data, b.ctypes.data if want_bias else None))
        return (v, b) if want_bias else v

    def set_weights(self, layer, values=None, bias=None):
        v = None if values is None else _np(values, np.float32)
        b = None if bias is None else _np(bias, np.float32)
        self._check(self._lib.sdnn_set_weights(self._h, layer, _addr(v), _addr(b)))

    def get_activations(self, layer, B):
        out = np.empty((B, self.n_neurons), dtype=np.float32)
        self._check(self._lib.sdnn_get_activations(self._h, layer, out.ctypes.data))
        return out

    def get_delta(self, layer, B):
        out = np.empty((B, self.n_neurons), dtype=np.float32)
        self._check(self._lib.sdnn_get_delta(self._h, layer, out.ctypes.data))
        return out

    def get_gradient(self, layer):
        out = np.empty(self.nnz[layer - 1], dtype=np.float32)
        self._check(self._lib.sdnn_get_gradient(self._h, layer, out.ctypes.data))
        return out

    def mirror_mismatches(self, layer):
        """Entries of the layer's transposed copy whose bits differ from the row-major copy (0 when consistent)."""
        c = ctypes.c_int64(0)
        self._check(self._lib.sdnn_mirror_mismatches(self._h, layer, ctypes.byref(c)))
        return c.value

    def get_phase_times(self):
        """(forward_ms, backward_ms) of the most recent train step."""
        a, b = ctypes.c_float(0.0), ctypes.c_float(0.0)
        self._check(self._lib.sdnn_get_phase_times(self._h, ctypes.byref(a), ctypes.byref(b)))
        return a.value, b.value

    def get_liveness(self):
        out = np.empty(self.n_layers, dtype=np.int32)
        self._check(self._lib.sdnn_get_liveness(self._h, out.ctypes.data))
        return out

    def infer_tile_width(self):
        """Inputs per tile that infer_batch uses on this handle."""
        return int(self._lib.sdnn_infer_tile_width(self._h))

    def infer_tiles_in_flight(self):
        """Tiles infer_batch keeps in flight on this handle when a batch has several (1 or 2)."""
        return int(self._lib.sdnn_infer_tiles_in_flight(self._h))

    def grouped_layers(self):
        """Layers for which FLAG_REORDER found groups of rows sharing a window of columns."""
        return int(self._lib.sdnn_grouped_layers(self._h))

    def windowed_layers(self):
        """Layers that run with their operand window staged in shared memory (FLAG_REORDER)."""
        return int(self._lib.sdnn_windowed_layers(self._h))

    def kernel_launches(self):
        return int(self._lib.sdnn_kernel_launches(self._h))

    def device_bytes(self):
        return int(self._lib.sdnn_device_bytes(self._h))

    def destroy(self):
        if self._h:
            self._lib.sdnn_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

"""Thin ctypes binding of libpatconv: argument marshalling only.

Every step of the layer runs inside the CUDA library.  There is no CPU
fallback: if the shared library cannot be loaded the import of this module's
functions fails loudly.  PyTorch appears only at the call sites (device memory
and streams); this module itself needs numpy and ctypes.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

from . import build as _build

F32, F16_F32ACC, I8_I32 = 0, 1, 2
DTYPES = {"f32": F32, "f16": F16_F32ACC, "i8": I8_I32}
OK = 0
STATIC_SCRATCH_BYTES = 8 << 20
STATUS_NAMES = {0: "OK", 1: "INVALID_ARG", 2: "BAD_PATTERN", 3: "SHAPE", 4: "UNSUPPORTED",
                5: "ALLOC", 6: "CUDA", 7: "TIMEOUT"}

EXPORTS = ["xgen_patconv_pack", "xgen_patconv_run", "xgen_patconv_run_static_scratch",
           "xgen_patconv_run_host", "xgen_patconv_enqueue_host", "xgen_patconv_plan",
           "xgen_patconv_plan_tuned", "xgen_patconv_plan_info", "xgen_patconv_test_expect_arrivals",
           "xgen_patconv_out_shape", "xgen_patconv_query", "xgen_patconv_view",
           "xgen_patconv_last_status", "xgen_patconv_free", "xgen_strerror",
           "xgen_patconv_launch_count", "xgen_patconv_probe", "xgen_patconv_run_fused",
           "xgen_blockgemm_pack", "xgen_blockgemm_run", "xgen_blockgemm_query", "xgen_blockgemm_view",
           "xgen_blockgemm_free",
           "xgen_dwconv_pack", "xgen_dwconv_run", "xgen_dwconv_query", "xgen_dwconv_free"]


class Desc(ctypes.Structure):
    _fields_ = [("c_in", ctypes.c_int32), ("c_out", ctypes.c_int32), ("stride", ctypes.c_int32),
                ("pad", ctypes.c_int32), ("dtype", ctypes.c_int), ("num_patterns", ctypes.c_int32),
                ("pattern_masks", ctypes.c_void_p)]


class Stats(ctypes.Structure):
    _fields_ = [("kernels_total", ctypes.c_int64), ("kernels_surviving", ctypes.c_int64),
                ("macs_per_pixel", ctypes.c_int64), ("weight_bytes", ctypes.c_int64),
                ("index_bytes", ctypes.c_int64), ("compact_index_bytes", ctypes.c_int64),
                ("csr_index_bytes", ctypes.c_int64),
                ("stream_bytes", ctypes.c_int64),
                ("filters_per_group", ctypes.c_int32), ("groups_per_block", ctypes.c_int32),
                ("n_blocks", ctypes.c_int32), ("channels_per_chunk", ctypes.c_int32),
                ("n_chunks", ctypes.c_int32), ("patterns_compiled", ctypes.c_int32),
                ("max_segment_slots", ctypes.c_int32),
                ("load_commands", ctypes.c_int64), ("group_imbalance", ctypes.c_double)]


class Tuning(ctypes.Structure):
    _fields_ = [("splits", ctypes.c_int32), ("no_copy_engine", ctypes.c_int32),
                ("no_launch_overlap", ctypes.c_int32), ("wait_limit_ms", ctypes.c_int32),
                ("no_small_blocks", ctypes.c_int32), ("reduce_mode", ctypes.c_int32),
                ("channels_per_chunk", ctypes.c_int32), ("groups_per_block", ctypes.c_int32)]


class PlanStats(ctypes.Structure):
    _fields_ = [("splits", ctypes.c_int32), ("chunks_per_split", ctypes.c_int32), ("tiles", ctypes.c_int32),
                ("filter_blocks", ctypes.c_int32), ("items", ctypes.c_int32), ("whole_items", ctypes.c_int32),
                ("blocks", ctypes.c_int32),
                ("threads_per_block", ctypes.c_int32), ("row_tiling", ctypes.c_int32),
                ("lanes_x", ctypes.c_int32), ("lanes_y", ctypes.c_int32),
                ("lanes_n", ctypes.c_int32), ("pixels_per_lane", ctypes.c_int32), ("stages", ctypes.c_int32),
                ("uses_copy_engine", ctypes.c_int32), ("shared_bytes", ctypes.c_int64),
                ("workspace_bytes", ctypes.c_int64), ("covered", ctypes.c_double),
                ("last_arriver", ctypes.c_int32), ("reserved", ctypes.c_int32)]


class ProbeResult(ctypes.Structure):
    _fields_ = [("ffma_tflops", ctypes.c_double), ("ffma2_tflops", ctypes.c_double), ("dp4a_tmacs", ctypes.c_double),
                ("launch_floor_us", ctypes.c_double), ("single_launch_us", ctypes.c_double),
                ("sm_count", ctypes.c_int32), ("sm_clock_mhz", ctypes.c_int32)]


class Epilogue(ctypes.Structure):
    _fields_ = [("relu", ctypes.c_int32), ("pool", ctypes.c_int32), ("residual_dev", ctypes.c_void_p),
                ("requant_scale_dev", ctypes.c_void_p), ("requant_zero_point", ctypes.c_int32)]


class GemmDesc(ctypes.Structure):
    _fields_ = [("k", ctypes.c_int32), ("c_out", ctypes.c_int32), ("block_rows", ctypes.c_int32),
                ("block_cols", ctypes.c_int32), ("dtype", ctypes.c_int), ("warps_per_block", ctypes.c_int32)]


class GemmStats(ctypes.Structure):
    _fields_ = [("weights_total", ctypes.c_int64), ("weights_kept", ctypes.c_int64),
                ("weight_bytes", ctypes.c_int64), ("stream_bytes", ctypes.c_int64),
                ("padded_slots", ctypes.c_int64), ("column_groups", ctypes.c_int64),
                ("row_commands", ctypes.c_int64), ("rows_per_warp", ctypes.c_int32),
                ("warps_per_block", ctypes.c_int32), ("row_blocks", ctypes.c_int32),
                ("stage_cols", ctypes.c_int32), ("n_stages", ctypes.c_int32),
                ("max_stage_bytes", ctypes.c_int32)]


class DwDesc(ctypes.Structure):
    _fields_ = [("channels", ctypes.c_int32), ("stride", ctypes.c_int32), ("pad", ctypes.c_int32),
                ("dtype", ctypes.c_int), ("num_patterns", ctypes.c_int32), ("pattern_masks", ctypes.c_void_p)]


class GemmHostView(ctypes.Structure):
    _fields_ = [("units", ctypes.c_void_p), ("n_units", ctypes.c_int64), ("seg_off", ctypes.c_void_p)]


class HostView(ctypes.Structure):
    _fields_ = [("slots", ctypes.c_void_p), ("n_slots", ctypes.c_int64),
                ("seg_off", ctypes.c_void_p), ("slot_oc", ctypes.c_void_p),
                ("compiled_masks", ctypes.c_void_p)]


class PatconvError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        super().__init__("%s failed: %s (%d)" % (where, STATUS_NAMES.get(status, "?"), status))


_lib = None


def lib():
    """Load libpatconv.so (building it first if it is missing or stale)."""
    global _lib
    if _lib is None:
        path = os.environ.get("XGEN_PATCONV_LIB") or _build.LIB_PATH    # another build of the library, if named
        if not os.path.exists(path):
            path = _build.build()
        L = ctypes.CDLL(path)
        P, I = ctypes.c_void_p, ctypes.c_int32
        L.xgen_patconv_pack.argtypes = [ctypes.POINTER(Desc), P, P, ctypes.c_int, ctypes.POINTER(P)]
        L.xgen_patconv_run.argtypes = [P, P, I, I, I, P, I, P, P]
        L.xgen_patconv_run_static_scratch.argtypes = [P, P, I, I, I, P, I, P, I, P]
        L.xgen_patconv_run_fused.argtypes = [P, P, I, I, I, P, ctypes.POINTER(Epilogue), P, P]
        L.xgen_patconv_run_host.argtypes = [P, P, I, I, I, P, I, P]
        L.xgen_patconv_enqueue_host.argtypes = [P, P, I, I, I, P, I, P, P]
        L.xgen_patconv_plan.argtypes = [P, I, I, I]
        L.xgen_patconv_plan_tuned.argtypes = [P, I, I, I, ctypes.POINTER(Tuning)]
        L.xgen_patconv_plan_info.argtypes = [P, I, I, I, ctypes.POINTER(PlanStats)]
        L.xgen_patconv_test_expect_arrivals.argtypes = [P, I]
        L.xgen_patconv_out_shape.argtypes = [P, I, I, ctypes.POINTER(I), ctypes.POINTER(I)]
        L.xgen_patconv_query.argtypes = [P, ctypes.POINTER(Stats)]
        L.xgen_patconv_view.argtypes = [P, ctypes.POINTER(HostView)]
        L.xgen_patconv_last_status.argtypes = [P, P]
        L.xgen_patconv_free.argtypes = [P]
        L.xgen_patconv_free.restype = None
        L.xgen_strerror.argtypes = [ctypes.c_int]
        L.xgen_strerror.restype = ctypes.c_char_p
        L.xgen_patconv_launch_count.restype = ctypes.c_int64
        L.xgen_patconv_probe.argtypes = [ctypes.c_int, ctypes.POINTER(ProbeResult)]
        L.xgen_blockgemm_pack.argtypes = [ctypes.POINTER(GemmDesc), P, P, P, ctypes.c_int, ctypes.POINTER(P)]
        L.xgen_blockgemm_run.argtypes = [P, P, ctypes.c_int64, P, I, P, P]
        L.xgen_blockgemm_query.argtypes = [P, ctypes.POINTER(GemmStats)]
        L.xgen_blockgemm_view.argtypes = [P, ctypes.POINTER(GemmHostView)]
        L.xgen_blockgemm_free.argtypes = [P]
        L.xgen_blockgemm_free.restype = None
        L.xgen_dwconv_pack.argtypes = [ctypes.POINTER(DwDesc), P, P, ctypes.c_int, ctypes.POINTER(P)]
        L.xgen_dwconv_run.argtypes = [P, P, I, I, I, P, I, P, P]
        L.xgen_dwconv_query.argtypes = [P, ctypes.POINTER(ctypes.c_int64)]
        L.xgen_dwconv_free.argtypes = [P]
        L.xgen_dwconv_free.restype = None
        for name in EXPORTS:
            if name not in ("xgen_patconv_free", "xgen_strerror", "xgen_patconv_launch_count", "xgen_blockgemm_free",
                            "xgen_dwconv_free"):
                getattr(L, name).restype = ctypes.c_int
        _lib = L
    return _lib


def _check(status, where):
    if status != OK:
        raise PatconvError(status, where)


class Packed:
    """Owner of one xgen_patconv_packed handle."""

    def __init__(self, c_in, c_out, stride, dtype, masks, dense_w, pattern_id, device=0, pad=1):
        self._h = ctypes.c_void_p()
        self.dtype = DTYPES[dtype] if isinstance(dtype, str) else int(dtype)
        self.c_in, self.c_out, self.stride = int(c_in), int(c_out), int(stride)
        masks = np.ascontiguousarray(masks, dtype=np.uint16)
        want = {F32: np.float32, F16_F32ACC: np.float16, I8_I32: np.int8}[self.dtype]
        w = np.ascontiguousarray(dense_w, dtype=want)
        pid = np.ascontiguousarray(pattern_id, dtype=np.int16)
        if w.size != c_out * c_in * 9 or pid.size != c_out * c_in:
            raise ValueError("dense_w must be [c_out,c_in,3,3] and pattern_id [c_out,c_in]")
        d = Desc(c_in, c_out, stride, pad, self.dtype, len(masks), masks.ctypes.data)
        _check(lib().xgen_patconv_pack(ctypes.byref(d), w.ctypes.data, pid.ctypes.data, int(device),
                                       ctypes.byref(self._h)), "xgen_patconv_pack")

    def close(self):
        if self._h:
            lib().xgen_patconv_free(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def out_shape(self, h, w):
        ho, wo = ctypes.c_int32(), ctypes.c_int32()
        _check(lib().xgen_patconv_out_shape(self._h, h, w, ctypes.byref(ho), ctypes.byref(wo)),
               "xgen_patconv_out_shape")
        return ho.value, wo.value

    def stats(self) -> dict:
        s = Stats()
        _check(lib().xgen_patconv_query(self._h, ctypes.byref(s)), "xgen_patconv_query")
        return {k: getattr(s, k) for k, _ in Stats._fields_}

    def view(self) -> dict:
        """Copies of the packed host arrays (see xgen_patconv_host_view)."""
        v = HostView()
        _check(lib().xgen_patconv_view(self._h, ctypes.byref(v)), "xgen_patconv_view")
        st = self.stats()
        J, G = st["filters_per_group"], st["groups_per_block"]
        nb, nc, npc = st["n_blocks"], st["n_chunks"], st["patterns_compiled"]

        def arr(ptr, n, ct, dt):
            if n == 0:
                return np.zeros(0, dt)
            return np.ctypeslib.as_array(ctypes.cast(ptr, ctypes.POINTER(ct)), shape=(n,)).astype(dt, copy=True)

        return {
            "slots": arr(v.slots, v.n_slots * 8, ctypes.c_uint32, np.uint32).reshape(-1, 8),
            "seg_off": arr(v.seg_off, nb * nc * (G + 1), ctypes.c_int32, np.int32).reshape(nb, nc, G + 1),
            "slot_oc": arr(v.slot_oc, nb * G * J, ctypes.c_int32, np.int32).reshape(nb, G, J),
            "masks": arr(v.compiled_masks, npc, ctypes.c_uint16, np.uint16),
        }

    def plan(self, n, h, w, splits=0, no_copy_engine=False, no_launch_overlap=False, wait_limit_ms=0,
             no_small_blocks=False, reduce_mode=0, channels_per_chunk=0, groups_per_block=0):
        """xgen_patconv_plan, or xgen_patconv_plan_tuned when any tuning field is given."""
        if (splits or no_copy_engine or no_launch_overlap or wait_limit_ms or no_small_blocks or reduce_mode
                or channels_per_chunk or groups_per_block):
            t = Tuning(int(splits), int(bool(no_copy_engine)), int(bool(no_launch_overlap)), int(wait_limit_ms),
                       int(bool(no_small_blocks)), int(reduce_mode), int(channels_per_chunk), int(groups_per_block))
            _check(lib().xgen_patconv_plan_tuned(self._h, n, h, w, ctypes.byref(t)), "xgen_patconv_plan_tuned")
        else:
            _check(lib().xgen_patconv_plan(self._h, n, h, w), "xgen_patconv_plan")

    def plan_info(self, n, h, w) -> dict:
        s = PlanStats()
        _check(lib().xgen_patconv_plan_info(self._h, n, h, w, ctypes.byref(s)), "xgen_patconv_plan_info")
        return {k: getattr(s, k) for k, _ in PlanStats._fields_ if k != "reserved"}

    def test_expect_arrivals(self, extra):
        _check(lib().xgen_patconv_test_expect_arrivals(self._h, int(extra)), "xgen_patconv_test_expect_arrivals")

    def run(self, x_ptr, n, h, w, bias_ptr, relu, y_ptr, stream=0):
        """Enqueue the layer; all pointers are device addresses (ints)."""
        _check(lib().xgen_patconv_run(self._h, x_ptr, n, h, w, bias_ptr or None, int(bool(relu)),
                                      y_ptr, stream or None), "xgen_patconv_run")

    def run_fused(self, x_ptr, n, h, w, bias_ptr, y_ptr, stream=0, relu=False, pool=0, residual_ptr=0,
                  requant_scale_ptr=0, zero_point=0):
        """xgen_patconv_run_fused: the layer with a residual addition, ReLU, a 2x2 max-pool and
        (integer layers) a re-quantisation to uint8 fused behind it; device addresses as ints."""
        ep = Epilogue(int(bool(relu)), int(pool), residual_ptr or None, requant_scale_ptr or None, int(zero_point))
        _check(lib().xgen_patconv_run_fused(self._h, x_ptr, n, h, w, bias_ptr or None, ctypes.byref(ep), y_ptr,
                                            stream or None), "xgen_patconv_run_fused")

    def run_static_scratch(self, x_ptr, n, h, w, bias_ptr, relu, y_ptr, splits, stream=0):
        """Like run(), with the channel chunks split `splits` ways and the partial sums kept
        in the library's built-in scratch array: no device memory is allocated.  For callers
        that may not allocate where they call; see the header for the size limit."""
        _check(lib().xgen_patconv_run_static_scratch(self._h, x_ptr, n, h, w, bias_ptr or None,
                                                     int(bool(relu)), y_ptr, int(splits), stream or None),
               "xgen_patconv_run_static_scratch")

    def run_host(self, x: np.ndarray, bias, relu) -> np.ndarray:
        """Host tensors in, host tensor out (copies inside the library)."""
        n, h, w, c = x.shape
        assert c == self.c_in and x.flags["C_CONTIGUOUS"]
        ho, wo = self.out_shape(h, w)
        ydt = {F32: np.float32, F16_F32ACC: np.float16, I8_I32: np.int32}[self.dtype]
        y = np.empty((n, ho, wo, self.c_out), dtype=ydt)
        b = None
        if bias is not None:
            b = np.ascontiguousarray(bias, dtype=np.int32 if self.dtype == I8_I32 else np.float32)
        _check(lib().xgen_patconv_run_host(self._h, x.ctypes.data, n, h, w,
                                           None if b is None else b.ctypes.data, int(bool(relu)),
                                           y.ctypes.data), "xgen_patconv_run_host")
        return y

    def enqueue_host_ptr(self, x_ptr, n, h, w, bias_ptr, relu, y_ptr, stream=0):
        """xgen_patconv_enqueue_host on raw host addresses (pinned buffers) and a raw
        cudaStream_t; returns without waiting, sync(stream) waits."""
        _check(lib().xgen_patconv_enqueue_host(self._h, x_ptr, n, h, w, bias_ptr or None, int(bool(relu)), y_ptr,
                                               stream or None), "xgen_patconv_enqueue_host")

    def run_host_ptr(self, x_ptr, n, h, w, bias_ptr, relu, y_ptr):
        """xgen_patconv_run_host on raw host addresses (e.g. pinned buffers)."""
        _check(lib().xgen_patconv_run_host(self._h, x_ptr, n, h, w, bias_ptr or None, int(bool(relu)), y_ptr),
               "xgen_patconv_run_host")

    def sync(self, stream=0):
        _check(lib().xgen_patconv_last_status(self._h, stream or None), "xgen_patconv_last_status")


def launch_count() -> int:
    return int(lib().xgen_patconv_launch_count())


def probe(device=0) -> dict:
    """xgen_patconv_probe: measured pipe rates and launch floor of the device."""
    r = ProbeResult()
    _check(lib().xgen_patconv_probe(int(device), ctypes.byref(r)), "xgen_patconv_probe")
    return {k: getattr(r, k) for k, _ in ProbeResult._fields_}


def strerror(status: int) -> str:
    return lib().xgen_strerror(int(status)).decode()


class BlockGemm:
    """Owner of one xgen_blockgemm_packed handle (block-pruned matrix product)."""

    def __init__(self, k, c_out, block_rows, block_cols, dtype, dense_w, row_keep, col_keep, device=0,
                 warps_per_block=0):
        self._h = ctypes.c_void_p()
        self.dtype = DTYPES[dtype] if isinstance(dtype, str) else int(dtype)
        self.k, self.c_out = int(k), int(c_out)
        want = {F32: np.float32, F16_F32ACC: np.float16}.get(self.dtype, np.float32)
        w = np.ascontiguousarray(dense_w, dtype=want)
        nbr, nbc = -(-c_out // block_rows), -(-k // block_cols)
        rk = np.ascontiguousarray(row_keep, dtype=np.uint8)
        ck = np.ascontiguousarray(col_keep, dtype=np.uint8)
        if w.size != c_out * k or rk.size != nbr * nbc * block_rows or ck.size != nbr * nbc * block_cols:
            raise ValueError("dense_w must be [c_out,k], row_keep [nbr,nbc,block_rows], col_keep [nbr,nbc,block_cols]")
        d = GemmDesc(k, c_out, block_rows, block_cols, self.dtype, int(warps_per_block))
        _check(lib().xgen_blockgemm_pack(ctypes.byref(d), w.ctypes.data, rk.ctypes.data, ck.ctypes.data, int(device),
                                         ctypes.byref(self._h)), "xgen_blockgemm_pack")

    def close(self):
        if self._h:
            lib().xgen_blockgemm_free(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def stats(self) -> dict:
        s = GemmStats()
        _check(lib().xgen_blockgemm_query(self._h, ctypes.byref(s)), "xgen_blockgemm_query")
        return {k: getattr(s, k) for k, _ in GemmStats._fields_}

    def view(self):
        """(units [n,4] uint32, seg_off int32): copies of the host image of the packed stream."""
        v = GemmHostView()
        _check(lib().xgen_blockgemm_view(self._h, ctypes.byref(v)), "xgen_blockgemm_view")
        st = self.stats()
        n_seg = st["row_blocks"] * st["n_stages"] * (st["warps_per_block"] + 1)
        units = np.ctypeslib.as_array(ctypes.cast(v.units, ctypes.POINTER(ctypes.c_uint32)), shape=(max(v.n_units, 0) * 4,)).copy() \
            if v.n_units > 0 else np.zeros(0, np.uint32)
        seg = np.ctypeslib.as_array(ctypes.cast(v.seg_off, ctypes.POINTER(ctypes.c_int32)), shape=(n_seg,)).copy()
        return units.reshape(-1, 4), seg

    def run(self, x_ptr, m, bias_ptr, relu, y_ptr, stream=0):
        """Enqueue the layer on a CUDA stream; pointers are device addresses (ints)."""
        _check(lib().xgen_blockgemm_run(self._h, ctypes.c_void_p(x_ptr), int(m), ctypes.c_void_p(bias_ptr or None),
                                        int(bool(relu)), ctypes.c_void_p(y_ptr), ctypes.c_void_p(stream or None)),
               "xgen_blockgemm_run")


class Depthwise:
    """Owner of one xgen_dwconv_packed handle (depthwise pattern-pruned 3x3 layer)."""

    def __init__(self, channels, stride, dtype, masks, dense_w, pattern_id, device=0, pad=1):
        self._h = ctypes.c_void_p()
        self.dtype = DTYPES[dtype] if isinstance(dtype, str) else int(dtype)
        self.c, self.stride = int(channels), int(stride)
        masks = np.ascontiguousarray(masks, dtype=np.uint16)
        want = {F32: np.float32, F16_F32ACC: np.float16}.get(self.dtype, np.float32)
        w = np.ascontiguousarray(dense_w, dtype=want)
        pid = np.ascontiguousarray(pattern_id, dtype=np.int16)
        if w.size != channels * 9 or pid.size != channels:
            raise ValueError("dense_w must be [channels,3,3] and pattern_id [channels]")
        d = DwDesc(channels, stride, pad, self.dtype, len(masks), masks.ctypes.data)
        _check(lib().xgen_dwconv_pack(ctypes.byref(d), w.ctypes.data, pid.ctypes.data, int(device),
                                      ctypes.byref(self._h)), "xgen_dwconv_pack")

    def close(self):
        if self._h:
            lib().xgen_dwconv_free(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def kernels_surviving(self) -> int:
        v = ctypes.c_int64()
        _check(lib().xgen_dwconv_query(self._h, ctypes.byref(v)), "xgen_dwconv_query")
        return v.value

    def run(self, x_ptr, n, h, w, bias_ptr, relu, y_ptr, stream=0):
        """Enqueue the layer on a CUDA stream; pointers are device addresses (ints)."""
        _check(lib().xgen_dwconv_run(self._h, ctypes.c_void_p(x_ptr), n, h, w, ctypes.c_void_p(bias_ptr or None),
                                     int(bool(relu)), ctypes.c_void_p(y_ptr), ctypes.c_void_p(stream or None)),
               "xgen_dwconv_run")

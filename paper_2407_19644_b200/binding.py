"""ctypes binding for libubp_b200.so. Names follow include/ubp.h."""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# UBP_B200_LIBRARY names another build of the same library to load instead (the checked build, libubp_b200_debug.so)
_LIB_PATH = os.environ.get("UBP_B200_LIBRARY") or os.path.join(_HERE, "libubp_b200.so")
_lib = None


class UbpError(RuntimeError):
    def __init__(self, code: int, what: str, msg: str = ""):
        super().__init__(f"{what} failed: {msg or code} ({code})")
        self.code = code


class _View(C.Structure):
    _fields_ = [("M", C.c_int32), ("C", C.c_int32), ("R", C.c_int32), ("Nb", C.c_int32), ("m", C.c_int32),
                ("indptr", C.POINTER(C.c_int32)), ("indices", C.POINTER(C.c_int32)), ("values", C.POINTER(C.c_float))]


class _PlanInfo(C.Structure):
    _fields_ = [("M", C.c_int32), ("C", C.c_int32), ("R", C.c_int32), ("Nb", C.c_int32), ("m", C.c_int32),
                ("variant", C.c_int32), ("panel_rows", C.c_int32), ("k_tile", C.c_int32),
                ("entries", C.c_int64), ("dev_bytes", C.c_int64)]


def lib_path() -> str:
    return _LIB_PATH


def load():
    """Load the shared library (once). Raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise RuntimeError(f"{_LIB_PATH} is missing: build it with `python -m paper_2407_19644_b200.build` "
                           "(there is no fallback implementation)")
    L = C.CDLL(_LIB_PATH)
    vp, sz, i32, i64 = C.c_void_p, C.c_size_t, C.c_int, C.c_int64
    L.ubp_strerror.restype = C.c_char_p
    L.ubp_strerror.argtypes = [i32]
    L.ubp_last_cuda_error.restype = i32
    L.ubp_pack.argtypes = [vp, vp, i32, i32, i32, i32, vp, sz, C.POINTER(sz)]
    L.ubp_unpack.argtypes = [vp, sz, vp, vp]
    L.ubp_blob_view.argtypes = [vp, sz, C.POINTER(_View)]
    L.ubp_variant_count.restype = i32
    L.ubp_variant_at.argtypes = [i32]
    L.ubp_variant_at.restype = i32
    L.ubp_variant_describe.argtypes = [i32, C.c_char_p, sz]
    L.ubp_plan_size.argtypes = [vp, sz, i32, C.POINTER(sz)]
    L.ubp_plan_image.argtypes = [vp, sz, i32, vp, sz, C.POINTER(C.c_int32)]
    L.ubp_plan_build.argtypes = [vp, sz, i32, vp, sz, vp, C.POINTER(vp)]
    L.ubp_plan_free.argtypes = [vp]
    L.ubp_plan_free.restype = None
    L.ubp_plan_info.argtypes = [vp, C.POINTER(_PlanInfo)]
    L.ubp_plan_check.argtypes = [vp, vp]
    L.ubp_plan_tile_choice.argtypes = [vp, i64, i32, C.POINTER(i32), C.POINTER(i32), C.POINTER(i32)]
    L.ubp_plan_tile_choice_conv.argtypes = [vp, i32, i32, i32, i32, C.POINTER(i32), C.POINTER(i32), C.POINTER(i32)]
    L.ubp_spmm.argtypes = [vp, vp, i64, i64, vp, i32, vp, i64, vp]
    L.ubp_conv1x1.argtypes = [vp, vp, i32, i32, i32, i64, i64, vp, i32, vp, i64, i64, vp]
    L.ubp_conv3x3_implicit.argtypes = [vp, vp, i32, i32, i32, i64, i64, vp, i32, vp, i64, i64, vp]
    L.ubp_plan_clear_status.argtypes = [vp, vp]
    L.ubp_selftest_bounded_wait.argtypes = [vp, C.c_uint, vp]
    L.ubp_static_plan_capacity.restype = sz
    L.ubp_spmm_static.argtypes = [vp, sz, vp, i64, i64, vp, i32, vp, i64, vp]
    L.ubp_conv3x3_strided.argtypes = [vp, vp, i32, i32, i32, i32, i64, i64, vp, i32, vp, i64, i64, vp]
    L.ubp_conv3x3_strided_scratch.restype = sz
    L.ubp_conv3x3_strided_scratch.argtypes = [i32, i32, i32, i32, i32]
    L.ubp_conv3x3_strided_ws.argtypes = [vp, vp, i32, i32, i32, i32, i64, i64, vp, sz, vp, i32, vp, i64, i64, vp]
    L.ubp_conv1x1_strided_scratch.restype = sz
    L.ubp_conv1x1_strided_scratch.argtypes = [i32, i32, i32, i32, i32]
    L.ubp_conv1x1_strided.argtypes = [vp, vp, i32, i32, i32, i32, i64, i64, vp, sz, vp, i32, vp, i64, i64, vp]
    L.ubp_pack_kmajor.argtypes = [vp, vp, i32, i32, i32, vp, sz, C.POINTER(sz)]
    L.ubp_kmajor_to_plan_blob.argtypes = [vp, sz, vp, sz, C.POINTER(sz)]
    L.ubp_plan_size_kmajor.argtypes = [vp, sz, i32, C.POINTER(sz)]
    L.ubp_plan_image_kmajor.argtypes = [vp, sz, i32, vp, sz, C.POINTER(C.c_int32)]
    L.ubp_plan_build_kmajor.argtypes = [vp, sz, i32, vp, sz, vp, C.POINTER(vp)]
    L.ubp_bed_workspace_size.argtypes = [i32, i32, i32, C.POINTER(sz)]
    L.ubp_block_scores.argtypes = [vp, i32, i32, i32, i32, vp, sz, vp, vp]
    L.ubp_bed_select.argtypes = [vp, i32, i32, i32, i32, i64, vp, sz, vp, vp, vp]
    _lib = L
    return L


def _chk(rc: int, what: str):
    if rc != 0:
        L = load()
        msg = L.ubp_strerror(rc).decode()
        if rc == -5:
            msg += f" [cuda error {L.ubp_last_cuda_error()}]"
        raise UbpError(rc, what, msg)


def _np_ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


# ------------------------------------------------------------------ host: format
def ubp_pack(W: np.ndarray, mask: np.ndarray, Nb: int) -> bytes:
    """mask [M][C] (0/1) + W [M][C] or [M][C][R] -> canonical blob (bytes)."""
    L = load()
    mask = np.ascontiguousarray(mask, dtype=np.uint8)
    if mask.ndim != 2:
        raise ValueError("mask must be [M][C]")
    M, Cin = mask.shape
    W = np.ascontiguousarray(W, dtype=np.float32)
    if W.size % (M * Cin) != 0 or W.size == 0:
        raise ValueError("W must be [M][C][R]")
    R = W.size // (M * Cin)
    n = C.c_size_t(0)
    _chk(L.ubp_pack(_np_ptr(W), _np_ptr(mask), M, Cin, R, Nb, None, 0, C.byref(n)), "ubp_pack")
    buf = np.empty(n.value, np.uint8)
    _chk(L.ubp_pack(_np_ptr(W), _np_ptr(mask), M, Cin, R, Nb, _np_ptr(buf), n.value, C.byref(n)), "ubp_pack")
    return buf.tobytes()


def blob_view(blob: bytes):
    """Validated view of a blob: dict with M, C, R, Nb, m and numpy copies of the three arrays."""
    L = load()
    b = np.frombuffer(blob, np.uint8)
    v = _View()
    _chk(L.ubp_blob_view(_np_ptr(b), b.size, C.byref(v)), "ubp_blob_view")
    indptr = np.ctypeslib.as_array(v.indptr, shape=(v.M + 1,)).copy()
    indices = np.ctypeslib.as_array(v.indices, shape=(max(v.m, 1),))[:v.m].copy()
    values = np.ctypeslib.as_array(v.values, shape=(max(v.m * v.Nb * v.R, 1),))[:v.m * v.Nb * v.R].copy()
    return dict(M=v.M, C=v.C, R=v.R, Nb=v.Nb, m=v.m, indptr=indptr, indices=indices,
                values=values.reshape(v.m, v.Nb, v.R))


def ubp_unpack(blob: bytes) -> Tuple[np.ndarray, np.ndarray]:
    """blob -> (W [M][C][R] with zeros where pruned, mask [M][C])."""
    L = load()
    d = blob_view(blob)
    b = np.frombuffer(blob, np.uint8)
    W = np.empty((d["M"], d["C"], d["R"]), np.float32)
    mask = np.empty((d["M"], d["C"]), np.uint8)
    _chk(L.ubp_unpack(_np_ptr(b), b.size, _np_ptr(W), _np_ptr(mask)), "ubp_unpack")
    return W, mask


pack_ubp = ubp_pack
unpack_ubp = ubp_unpack


def ubp_pack_kmajor(W: np.ndarray, mask: np.ndarray, B: int) -> bytes:
    """Blocks of B consecutive input channels inside one output row: mask [M][C] + W [M][C] -> the canonical blob of
    the transposed layer."""
    L = load()
    mask = np.ascontiguousarray(mask, dtype=np.uint8)
    M, Cin = mask.shape
    W = np.ascontiguousarray(W, dtype=np.float32).reshape(M, Cin)
    n = C.c_size_t(0)
    _chk(L.ubp_pack_kmajor(_np_ptr(W), _np_ptr(mask), M, Cin, B, None, 0, C.byref(n)), "ubp_pack_kmajor")
    buf = np.empty(n.value, np.uint8)
    _chk(L.ubp_pack_kmajor(_np_ptr(W), _np_ptr(mask), M, Cin, B, _np_ptr(buf), n.value, C.byref(n)), "ubp_pack_kmajor")
    return buf.tobytes()


def ubp_kmajor_to_plan_blob(kblob: bytes) -> bytes:
    """Blob of ubp_pack_kmajor -> a blob Plan() accepts (the layer's own orientation, blocks of one output channel)."""
    L = load()
    b = np.frombuffer(kblob, np.uint8)
    n = C.c_size_t(0)
    _chk(L.ubp_kmajor_to_plan_blob(_np_ptr(b), b.size, None, 0, C.byref(n)), "ubp_kmajor_to_plan_blob")
    buf = np.empty(n.value, np.uint8)
    _chk(L.ubp_kmajor_to_plan_blob(_np_ptr(b), b.size, _np_ptr(buf), n.value, C.byref(n)), "ubp_kmajor_to_plan_blob")
    return buf.tobytes()


def variants():
    L = load()
    out = {}
    buf = C.create_string_buffer(256)
    for k in range(L.ubp_variant_count()):
        i = L.ubp_variant_at(k)
        _chk(L.ubp_variant_describe(i, buf, 256), "ubp_variant_describe")
        out[i] = buf.value.decode()
    return out


def plan_size(blob: bytes, variant: int = 0, kmajor: bool = False) -> int:
    """Bytes of device memory the plan needs. kmajor: `blob` comes from ubp_pack_kmajor (blocks along the input
    channels)."""
    L = load()
    b = np.frombuffer(blob, np.uint8)
    n = C.c_size_t(0)
    fn = L.ubp_plan_size_kmajor if kmajor else L.ubp_plan_size
    _chk(fn(_np_ptr(b), b.size, variant, C.byref(n)), "ubp_plan_size")
    return n.value


def plan_image(blob: bytes, variant: int = 0, kmajor: bool = False):
    """Host copy of the device plan image and its geometry (no GPU needed)."""
    L = load()
    b = np.frombuffer(blob, np.uint8)
    n = plan_size(blob, variant, kmajor)
    buf = np.zeros(n, np.uint8)
    geom = (C.c_int32 * 8)()
    fn = L.ubp_plan_image_kmajor if kmajor else L.ubp_plan_image
    _chk(fn(_np_ptr(b), b.size, variant, _np_ptr(buf), n, geom), "ubp_plan_image")
    keys = ["nbk", "panel_rows", "k_tile", "WR", "dupw", "nkt", "NP", "NG"]
    return buf, dict(zip(keys, [int(g) for g in geom]))


# ------------------------------------------------------------------ device
def _stream_ptr(stream=None):
    import torch
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _dev_ptr(t, name, allow_none=False):
    import torch
    if t is None:
        if allow_none:
            return None
        raise ValueError(f"{name} is required")
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == torch.float32):
        raise ValueError(f"{name} must be a float32 CUDA tensor")
    return C.c_void_p(t.data_ptr())


class Plan:
    """Device plan of one packed layer. The device buffer is a torch uint8
    tensor owned by this object; the library holds only a small host handle."""

    def __init__(self, blob: bytes, variant: int = 0, device="cuda", stream=None, kmajor: bool = False):
        """kmajor: `blob` comes from ubp_pack_kmajor (blocks of consecutive input channels inside one output row)."""
        import torch
        L = load()
        self._lib = L
        self._handle = None
        b = np.frombuffer(blob, np.uint8)
        n = plan_size(blob, variant, kmajor)
        self.buffer = torch.empty(n + 256, dtype=torch.uint8, device=device)
        base = self.buffer.data_ptr()
        self._dev = (base + 255) // 256 * 256
        h = C.c_void_p()
        with torch.cuda.device(self.buffer.device):
            build = L.ubp_plan_build_kmajor if kmajor else L.ubp_plan_build
            _chk(build(_np_ptr(b), b.size, variant, C.c_void_p(self._dev), n, _stream_ptr(stream), C.byref(h)),
                 "ubp_plan_build")
        self._handle = h
        info = _PlanInfo()
        _chk(L.ubp_plan_info(h, C.byref(info)), "ubp_plan_info")
        self.M, self.C, self.R, self.Nb, self.m = info.M, info.C, info.R, info.Nb, info.m
        self.variant, self.panel_rows, self.k_tile = info.variant, info.panel_rows, info.k_tile
        self.entries, self.dev_bytes = info.entries, info.dev_bytes

    @property
    def handle(self):
        if self._handle is None:
            raise RuntimeError("plan was freed")
        return self._handle

    def check(self, stream=None):
        """Synchronise the stream and raise if a kernel reported a failed bounded wait."""
        _chk(self._lib.ubp_plan_check(self.handle, _stream_ptr(stream)), "ubp_plan_check")

    def tile_choice(self, Nc: int, image_width: int = 0):
        """(kernel, tile_rows, tile_cols) of a fast-path launch over Nc columns on the plan's device (3x3 plans:
        Nc = batch * height * width and image_width = width; strided 3x3: Nc = batch * Ho * Wo and image_width = -width):
        kernel 0 = sparse FP32, 1 = tensor core / one CTA per tile, 2 = tensor core / CTA pair per tile, 3 = the
        comparison kernels that walk the canonical arrays."""
        k, r, c = C.c_int32(), C.c_int32(), C.c_int32()
        import torch
        with torch.cuda.device(self.buffer.device):
            _chk(self._lib.ubp_plan_tile_choice(self.handle, int(Nc), int(image_width), C.byref(k), C.byref(r), C.byref(c)),
                 "ubp_plan_tile_choice")
        return k.value, r.value, c.value

    def tile_choice_conv(self, B: int, H: int, Wd: int, stride: int = 1):
        """(kernel, tile_rows, tile_cols) of a fast-path 3x3 launch on B images of H x Wd pixels; kernel 4 = the CTA-pair
        kernel on the padded pixel grid (tile_cols in padded positions), else as tile_choice."""
        k, r, c = C.c_int32(), C.c_int32(), C.c_int32()
        import torch
        with torch.cuda.device(self.buffer.device):
            _chk(self._lib.ubp_plan_tile_choice_conv(self.handle, int(B), int(H), int(Wd), int(stride), C.byref(k), C.byref(r),
                                                     C.byref(c)), "ubp_plan_tile_choice_conv")
        return k.value, r.value, c.value

    def clear_status(self, stream=None):
        _chk(self._lib.ubp_plan_clear_status(self.handle, _stream_ptr(stream)), "ubp_plan_clear_status")

    def selftest_bounded_wait(self, limit_us: int = 20000, stream=None):
        """Launch the library's wait self test: a kernel whose wait can never complete gives up after `limit_us`
        and flags the plan; check() then raises UbpError(-7)."""
        _chk(self._lib.ubp_selftest_bounded_wait(self.handle, int(limit_us), _stream_ptr(stream)),
             "ubp_selftest_bounded_wait")

    def free(self):
        if self._handle is not None:
            self._lib.ubp_plan_free(self._handle)
            self._handle = None

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass


def ubp_spmm(plan: Plan, X, bias=None, relu: bool = False, out=None, stream=None):
    """Y[M][Nc] = act(Wm @ X + bias); X is a float32 CUDA tensor [C][Nc] whose rows may be strided."""
    import torch
    if X.dim() != 2 or X.shape[0] != plan.C or X.stride(1) != 1 and X.shape[1] > 1:
        raise ValueError("X must be [C][Nc] with unit column stride")
    Nc = X.shape[1]
    if out is None:
        out = torch.empty((plan.M, Nc), dtype=torch.float32, device=X.device)
    if out.shape != (plan.M, Nc) or (out.stride(1) != 1 and Nc > 1):
        raise ValueError("out must be [M][Nc] with unit column stride")
    with torch.cuda.device(X.device):
        _chk(plan._lib.ubp_spmm(plan.handle, _dev_ptr(X, "X"), X.stride(0), Nc, _dev_ptr(bias, "bias", True),
                                int(bool(relu)), _dev_ptr(out, "out"), out.stride(0), _stream_ptr(stream)), "ubp_spmm")
    return out


def _conv_args(plan, x, out, layout, stride=1):
    import torch
    if stride < 1:
        raise ValueError("stride must be >= 1")
    if layout == "CNHW":
        Cin, B, H, Wd = x.shape
        sb, sc = x.stride(1), x.stride(0)
        oshape = (plan.M, B, (H - 1) // stride + 1, (Wd - 1) // stride + 1)
    elif layout == "NCHW":
        B, Cin, H, Wd = x.shape
        sb, sc = x.stride(0), x.stride(1)
        oshape = (B, plan.M, (H - 1) // stride + 1, (Wd - 1) // stride + 1)
    else:
        raise ValueError("layout must be 'CNHW' or 'NCHW'")
    if Cin != plan.C or x.stride(3) != 1 or x.stride(2) != Wd:
        raise ValueError("input planes must be contiguous [H][W] and have plan.C channels")
    if out is None:
        out = torch.empty(oshape, dtype=torch.float32, device=x.device)
    if tuple(out.shape) != oshape or out.stride(3) != 1 or out.stride(2) != oshape[3]:
        raise ValueError("bad output tensor")
    osb, osc = (out.stride(1), out.stride(0)) if layout == "CNHW" else (out.stride(0), out.stride(1))
    return B, H, Wd, sb, sc, out, osb, osc


def ubp_conv1x1(plan: Plan, x, bias=None, relu: bool = False, out=None, layout: str = "CNHW", stream=None,
                stride: int = 1, scratch=None):
    """1x1 convolution. layout 'CNHW': x [C][B][H][W] -> out [M][B][Ho][Wo]; 'NCHW': x [B][C][H][W]. With stride > 1
    the pixels read are gathered into `scratch` first (a float32 CUDA tensor of at least C*B*Ho*Wo elements; allocated
    here when not given)."""
    import torch
    B, H, Wd, sb, sc, out, osb, osc = _conv_args(plan, x, out, layout, stride)
    if stride != 1:
        need = plan._lib.ubp_conv1x1_strided_scratch(plan.C, B, H, Wd, stride)
        if scratch is None:
            scratch = torch.empty(need // 4, dtype=torch.float32, device=x.device)
        with torch.cuda.device(x.device):
            _chk(plan._lib.ubp_conv1x1_strided(plan.handle, _dev_ptr(x, "x"), B, H, Wd, stride, sb, sc,
                                               _dev_ptr(scratch, "scratch"), scratch.numel() * 4,
                                               _dev_ptr(bias, "bias", True), int(bool(relu)), _dev_ptr(out, "out"),
                                               osb, osc, _stream_ptr(stream)), "ubp_conv1x1_strided")
            scratch.record_stream(torch.cuda.current_stream() if stream is None else stream)
        return out
    with torch.cuda.device(x.device):
        _chk(plan._lib.ubp_conv1x1(plan.handle, _dev_ptr(x, "x"), B, H, Wd, sb, sc, _dev_ptr(bias, "bias", True),
                                   int(bool(relu)), _dev_ptr(out, "out"), osb, osc, _stream_ptr(stream)), "ubp_conv1x1")
    return out


def ubp_conv3x3_implicit(plan: Plan, x, bias=None, relu: bool = False, out=None, layout: str = "CNHW", stream=None,
                         stride: int = 1, scratch=None):
    """3x3 / pad 1 convolution on a plan built from an R = 9 blob. stride 2: the four phase planes of the input go to
    `scratch` first (a float32 CUDA tensor of at least 4*C*B*Ho*Wo (+ row padding) elements; allocated here when not
    given), then the padded-grid kernel runs on them where the plan and layout allow; other strides > 1: the one-CTA
    tensor-core kernel or one lane per output pixel."""
    import torch
    B, H, Wd, sb, sc, out, osb, osc = _conv_args(plan, x, out, layout, stride)
    if stride != 1:
        need = plan._lib.ubp_conv3x3_strided_scratch(plan.C, B, H, Wd, stride)
        if scratch is None and need:
            scratch = torch.empty(need // 4, dtype=torch.float32, device=x.device)
        with torch.cuda.device(x.device):
            _chk(plan._lib.ubp_conv3x3_strided_ws(plan.handle, _dev_ptr(x, "x"), B, H, Wd, stride, sb, sc,
                                                  _dev_ptr(scratch, "scratch", True), scratch.numel() * 4 if scratch is not None else 0,
                                                  _dev_ptr(bias, "bias", True), int(bool(relu)), _dev_ptr(out, "out"),
                                                  osb, osc, _stream_ptr(stream)), "ubp_conv3x3_strided_ws")
            if scratch is not None:
                scratch.record_stream(torch.cuda.current_stream() if stream is None else stream)
        return out
    with torch.cuda.device(x.device):
        _chk(plan._lib.ubp_conv3x3_implicit(plan.handle, _dev_ptr(x, "x"), B, H, Wd, sb, sc,
                                            _dev_ptr(bias, "bias", True), int(bool(relu)), _dev_ptr(out, "out"),
                                            osb, osc, _stream_ptr(stream)), "ubp_conv3x3_implicit")
    return out


def ubp_spmm_static(blob: bytes, X, bias=None, relu: bool = False, out=None, stream=None):
    """ubp_spmm without a Plan object: for callers that must not allocate device memory.

    The plan is rebuilt from `blob` on the host and uploaded into the library's fixed 2 MiB device
    array on every call, so pass `out` (preallocated [M][Nc]) -- then nothing in this call allocates on the
    device. Calls whose GPU work could overlap share that array and must be serialised by the caller.
    Raises UbpError(-8) when the layer's plan does not fit the array."""
    import torch
    L = load()
    b = np.frombuffer(blob, np.uint8)
    d = blob_view(blob)
    if X.dim() != 2 or X.shape[0] != d["C"] or (X.stride(1) != 1 and X.shape[1] > 1):
        raise ValueError("X must be [C][Nc] with unit column stride")
    Nc = X.shape[1]
    if out is None:
        out = torch.empty((d["M"], Nc), dtype=torch.float32, device=X.device)
    if tuple(out.shape) != (d["M"], Nc) or (out.stride(1) != 1 and Nc > 1):
        raise ValueError("out must be [M][Nc] with unit column stride")
    with torch.cuda.device(X.device):
        _chk(L.ubp_spmm_static(_np_ptr(b), b.size, _dev_ptr(X, "X"), X.stride(0), Nc, _dev_ptr(bias, "bias", True),
                               int(bool(relu)), _dev_ptr(out, "out"), out.stride(0), _stream_ptr(stream)),
             "ubp_spmm_static")
    return out


def static_plan_capacity() -> int:
    return int(load().ubp_static_plan_capacity())


# ------------------------------------------------------------------ block selection (Section 4.1)
class BedSelector:
    """Device scratch for block selection on layers of one shape ([M][C][R] weights, block size Nb); the scratch
    is a torch uint8 tensor owned by this object, so repeated calls allocate nothing but their outputs."""

    def __init__(self, M: int, Cin: int, R: int, Nb: int, device="cuda"):
        import torch
        self._lib = load()
        self.M, self.C, self.R, self.Nb = int(M), int(Cin), int(R), int(Nb)
        n = C.c_size_t(0)
        _chk(self._lib.ubp_bed_workspace_size(self.M, self.C, self.Nb, C.byref(n)), "ubp_bed_workspace_size")
        self.bytes = n.value
        self.buffer = torch.empty(n.value + 256, dtype=torch.uint8, device=device)
        self._base = (self.buffer.data_ptr() + 255) // 256 * 256

    def _w(self, W):
        import torch
        if not (isinstance(W, torch.Tensor) and W.is_cuda and W.dtype == torch.float32 and W.is_contiguous()
                and W.numel() == self.M * self.C * self.R and W.shape[0] == self.M and W.shape[1] == self.C):
            raise ValueError("W must be a contiguous float32 CUDA tensor [M][C][R] of this selector's shape")
        if W.device != self.buffer.device:
            raise ValueError("W is on another device than the selector")
        return C.c_void_p(W.data_ptr())

    def scores(self, W, out=None, stream=None):
        """Eq. 1 scores of every candidate block: float32 CUDA tensor [C][M], -inf where the block would leave
        the weights."""
        import torch
        if out is None:
            out = torch.empty((self.C, self.M), dtype=torch.float32, device=W.device)
        with torch.cuda.device(W.device):
            _chk(self._lib.ubp_block_scores(self._w(W), self.M, self.C, self.R, self.Nb, C.c_void_p(self._base),
                                            self.bytes, C.c_void_p(out.data_ptr()), _stream_ptr(stream)),
                 "ubp_block_scores")
        return out

    def select(self, W, m: int, mask=None, n_selected=None, stream=None):
        """Block expansion and division: (mask uint8 CUDA tensor [M][C], n_selected int64 CUDA tensor [1])."""
        import torch
        if mask is None:
            mask = torch.empty((self.M, self.C), dtype=torch.uint8, device=W.device)
        if n_selected is None:
            n_selected = torch.zeros(1, dtype=torch.int64, device=W.device)
        if mask.dtype != torch.uint8 or tuple(mask.shape) != (self.M, self.C) or not mask.is_contiguous():
            raise ValueError("mask must be a contiguous uint8 CUDA tensor [M][C]")
        with torch.cuda.device(W.device):
            _chk(self._lib.ubp_bed_select(self._w(W), self.M, self.C, self.R, self.Nb, int(m), C.c_void_p(self._base),
                                          self.bytes, C.c_void_p(mask.data_ptr()), C.c_void_p(n_selected.data_ptr()),
                                          _stream_ptr(stream)), "ubp_bed_select")
        return mask, n_selected


def _selector_for(W, Nb: int) -> BedSelector:
    if W.dim() not in (2, 3):
        raise ValueError("W must be [M][C] or [M][C][R]")
    return BedSelector(W.shape[0], W.shape[1], W.shape[2] if W.dim() == 3 else 1, Nb, device=W.device)


def ubp_block_scores(W, Nb: int, stream=None):
    """One-shot form of BedSelector.scores (allocates its scratch; synchronises before freeing it)."""
    import torch
    sel = _selector_for(W, Nb)
    S = sel.scores(W, stream=stream)
    torch.cuda.synchronize(W.device)
    return S


def ubp_bed_select(W, Nb: int, m: int, stream=None):
    """One-shot form of BedSelector.select (allocates its scratch; synchronises before freeing it)."""
    import torch
    sel = _selector_for(W, Nb)
    out = sel.select(W, m, stream=stream)
    torch.cuda.synchronize(W.device)
    return out

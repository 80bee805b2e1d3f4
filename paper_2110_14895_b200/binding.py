"""ctypes binding of libvit_b200.so: the same entry points as include/vit.h, argument
marshalling only.  Every step of the forward pass runs in the library's CUDA kernels; there is
no fallback: if the library is missing or a call fails, an exception is raised.

PyTorch appears here only as the owner of device memory and streams (`data_ptr()`,
`torch.cuda.Stream.cuda_stream`).
"""
import ctypes
import os
from ctypes import (POINTER, Structure, byref, c_char_p, c_float, c_int, c_int32, c_size_t,
                    c_uint64, c_void_p)

import numpy as np

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libvit_b200.so")

VIT_OK = 0
VIT_ERR_INVALID_ARG, VIT_ERR_RANGE, VIT_ERR_CONFIG, VIT_ERR_WORKSPACE = -1, -2, -3, -4
VIT_ERR_CUDA, VIT_ERR_TIMEOUT, VIT_ERR_NO_DEVICE = -5, -6, -7
VIT_ERR_TOO_LARGE = -8
VIT_ERR_INFEASIBLE = -9
VIT_HEAD_STATIC_MAX_FLOATS = 512 * 1024
VIT_BF16, VIT_FP32 = 0, 1
VIT_TILING_AUTO, VIT_TILING_128x128, VIT_TILING_128x256, VIT_TILING_PAIR_256x256 = 0, 1, 2, 3

EXPORTS = [
    "vit_param_count", "vit_workspace_bytes", "vit_pipeline_workspace_bytes", "vit_create",
    "vit_destroy", "vit_patch_embed", "vit_run_stage", "vit_head", "vit_run_pipeline",
    "vit_run_pipeline_host", "vit_run_pipeline_grouped", "vit_check_status", "vit_launch_count", "vit_status_string",
    "vit_op_layernorm", "vit_op_linear", "vit_op_linear_tiled", "vit_op_attention", "vit_op_rowstats", "vit_op_linear_ln", "vit_profile_enable",
    "vit_profile_collect", "vit_head_static", "vit_partition", "vit_partition_categories",
    "vit_debug_wait_probe",
]
PROF_CLASSES = ["layernorm", "qkv", "attention", "outproj", "fc1", "fc2", "embed", "head", "op"]


class VitConfig(Structure):
    _fields_ = [
        ("image_size", c_int32), ("patch_size", c_int32), ("channels", c_int32),
        ("hidden", c_int32), ("layers", c_int32), ("heads", c_int32), ("mlp_dim", c_int32),
        ("num_classes", c_int32), ("ln_eps", c_float), ("dtype", c_int32),
        ("max_microbatch", c_int32), ("extra_tokens", c_int32),
    ]


class VitPartitionProblem(Structure):
    _fields_ = [
        ("layers", c_int32), ("devices", c_int32), ("layer_time", c_void_p), ("out_bytes", c_void_p),
        ("layer_mem", c_void_p), ("device_mem", c_void_p), ("bandwidth", c_void_p),
    ]


class VitError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


_lib = None


def lib():
    """Loads the shared library (once).  Fails loudly when it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2110_14895_b200.build`")
    L = ctypes.CDLL(LIB_PATH)
    P = POINTER
    L.vit_param_count.restype = c_size_t
    L.vit_param_count.argtypes = [P(VitConfig)]
    L.vit_workspace_bytes.restype = c_size_t
    L.vit_workspace_bytes.argtypes = [P(VitConfig), c_int]
    L.vit_pipeline_workspace_bytes.restype = c_size_t
    L.vit_pipeline_workspace_bytes.argtypes = [P(VitConfig), c_int]
    L.vit_create.restype = c_int
    L.vit_create.argtypes = [P(VitConfig), c_void_p, c_size_t, P(c_void_p)]
    L.vit_destroy.restype = c_int
    L.vit_destroy.argtypes = [c_void_p]
    L.vit_patch_embed.restype = c_int
    L.vit_patch_embed.argtypes = [c_void_p, c_int, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]
    L.vit_run_stage.restype = c_int
    L.vit_run_stage.argtypes = [c_void_p, c_int, c_int, c_int, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]
    L.vit_head.restype = c_int
    L.vit_head.argtypes = [c_void_p, c_int, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]
    for f in (L.vit_run_pipeline, L.vit_run_pipeline_host):
        f.restype = c_int
        f.argtypes = [c_void_p, P(c_int32), c_int, c_int, c_int, c_void_p, c_void_p, P(c_void_p),
                      c_size_t, P(c_void_p), c_int]
    L.vit_run_pipeline_grouped.restype = c_int
    L.vit_run_pipeline_grouped.argtypes = [c_void_p, P(c_int32), c_int, c_int, c_int, c_int, c_void_p, c_void_p,
                                           P(c_void_p), c_size_t, P(c_void_p), c_int]
    L.vit_check_status.restype = c_int
    L.vit_check_status.argtypes = [c_void_p, c_void_p]
    L.vit_launch_count.restype = c_uint64
    L.vit_launch_count.argtypes = [c_void_p]
    L.vit_status_string.restype = c_char_p
    L.vit_status_string.argtypes = [c_int]
    L.vit_op_layernorm.restype = c_int
    L.vit_op_layernorm.argtypes = [c_void_p, c_int, c_int, c_int, c_void_p, c_void_p, c_void_p, c_float, c_void_p, c_void_p]
    L.vit_op_linear.restype = c_int
    L.vit_op_linear.argtypes = [c_void_p, c_int, c_int, c_int, c_int, c_void_p, c_void_p, c_void_p, c_int, c_void_p, c_void_p, c_void_p]
    L.vit_op_linear_tiled.restype = c_int
    L.vit_op_linear_tiled.argtypes = [c_void_p, c_int, c_int, c_int, c_int, c_void_p, c_void_p, c_void_p, c_int, c_void_p, c_void_p, c_int, c_void_p]
    L.vit_op_rowstats.restype = c_int
    L.vit_op_rowstats.argtypes = [c_void_p, c_int, c_int, c_void_p, c_float, c_void_p, c_void_p]
    L.vit_op_linear_ln.restype = c_int
    L.vit_op_linear_ln.argtypes = [c_void_p, c_int, c_int, c_int, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p,
                                   c_int, c_void_p, c_int, c_void_p]
    L.vit_op_attention.restype = c_int
    L.vit_op_attention.argtypes = [c_void_p, c_int, c_int, c_int, c_int, c_int, c_void_p, c_void_p, c_void_p]
    L.vit_head_static.restype = c_int
    L.vit_head_static.argtypes = [c_void_p, c_int, c_void_p, c_void_p, c_void_p]
    L.vit_partition.restype = c_int
    L.vit_partition.argtypes = [P(VitPartitionProblem), P(ctypes.c_double), P(c_int32), c_void_p, c_void_p]
    L.vit_partition_categories.restype = c_int
    L.vit_partition_categories.argtypes = [P(VitPartitionProblem), c_void_p, P(ctypes.c_double), P(c_int32),
                                           c_void_p, c_void_p]
    L.vit_debug_wait_probe.restype = c_int
    L.vit_debug_wait_probe.argtypes = [c_void_p, ctypes.c_int64, c_void_p]
    L.vit_profile_enable.restype = c_int
    L.vit_profile_enable.argtypes = [c_void_p, c_int]
    L.vit_profile_collect.restype = c_int
    L.vit_profile_collect.argtypes = [c_void_p, P(ctypes.c_double), P(c_uint64)]
    _lib = L
    return L


def status_string(status: int) -> str:
    return lib().vit_status_string(status).decode()


def _check(status, where):
    if status != VIT_OK:
        raise VitError(status, where)


def make_config(shape, dtype=VIT_BF16, max_microbatch=1) -> VitConfig:
    """`shape` is any object with image_size, patch_size, channels, hidden, layers, heads,
    mlp_dim, num_classes, ln_eps attributes."""
    return VitConfig(shape.image_size, shape.patch_size, shape.channels, shape.hidden, shape.layers,
                     shape.heads, shape.mlp_dim, shape.num_classes, float(shape.ln_eps), int(dtype),
                     int(max_microbatch), int(getattr(shape, "extra_tokens", 0)))


# ---- thin wrappers with the names of the C entry points (raw pointers as ints) ----------------
def vit_param_count(cfg: VitConfig) -> int:
    return lib().vit_param_count(byref(cfg))


def vit_workspace_bytes(cfg: VitConfig, microbatch: int) -> int:
    return lib().vit_workspace_bytes(byref(cfg), microbatch)


def vit_pipeline_workspace_bytes(cfg: VitConfig, microbatch: int) -> int:
    return lib().vit_pipeline_workspace_bytes(byref(cfg), microbatch)


def vit_create(cfg: VitConfig, host_params: np.ndarray) -> int:
    if host_params.dtype != np.float32 or not host_params.flags["C_CONTIGUOUS"]:
        raise TypeError("host_params must be a contiguous float32 array")
    h = c_void_p()
    _check(lib().vit_create(byref(cfg), host_params.ctypes.data, host_params.size, byref(h)), "vit_create")
    return h.value


def vit_destroy(h: int) -> None:
    _check(lib().vit_destroy(h), "vit_destroy")


def vit_patch_embed(h, microbatch, pixels, tokens_out, ws, ws_bytes, stream=0):
    _check(lib().vit_patch_embed(h, microbatch, pixels, tokens_out, ws, ws_bytes, stream), "vit_patch_embed")


def vit_run_stage(h, layer_begin, layer_end, microbatch, inp, out, ws, ws_bytes, stream=0):
    _check(lib().vit_run_stage(h, layer_begin, layer_end, microbatch, inp, out, ws, ws_bytes, stream),
           "vit_run_stage")


def vit_head(h, microbatch, tokens, logits, ws, ws_bytes, stream=0):
    _check(lib().vit_head(h, microbatch, tokens, logits, ws, ws_bytes, stream), "vit_head")


def vit_head_static(h, microbatch, tokens, logits, stream=0):
    """vit_head with the scratch inside the library: for callers that cannot allocate device
    memory.  Raises VitError(VIT_ERR_TOO_LARGE) beyond microbatch * hidden = 512 Ki."""
    _check(lib().vit_head_static(h, microbatch, tokens, logits, stream), "vit_head_static")


def _pipeline(fn, name, h, stage_layers, batch, microbatch, pixels, logits, ws_ptrs, ws_bytes, streams):
    n = len(stage_layers)
    sl = (c_int32 * n)(*stage_layers)
    k = len(streams)
    if len(ws_ptrs) != k:
        raise ValueError("one workspace per stream")
    wsa = (c_void_p * k)(*ws_ptrs)
    sta = (c_void_p * k)(*streams)
    _check(fn(h, sl, n, batch, microbatch, pixels, logits, wsa, ws_bytes, sta, k), name)


def vit_run_pipeline(h, stage_layers, batch, microbatch, pixels, logits, ws_ptrs, ws_bytes, streams):
    _pipeline(lib().vit_run_pipeline, "vit_run_pipeline", h, stage_layers, batch, microbatch, pixels,
              logits, ws_ptrs, ws_bytes, streams)


def vit_run_pipeline_host(h, stage_layers, batch, microbatch, host_pixels, host_logits, ws_ptrs,
                          ws_bytes, streams):
    _pipeline(lib().vit_run_pipeline_host, "vit_run_pipeline_host", h, stage_layers, batch, microbatch,
              host_pixels, host_logits, ws_ptrs, ws_bytes, streams)


def vit_run_pipeline_grouped(h, stage_layers, batch, microbatch, group, pixels, logits, ws_ptrs, ws_bytes, streams):
    n = len(stage_layers)
    sl = (c_int32 * n)(*stage_layers)
    k = len(streams)
    if len(ws_ptrs) != k:
        raise ValueError("one workspace per stream")
    wsa = (c_void_p * k)(*ws_ptrs)
    sta = (c_void_p * k)(*streams)
    _check(lib().vit_run_pipeline_grouped(h, sl, n, batch, microbatch, group, pixels, logits, wsa, ws_bytes, sta, k),
           "vit_run_pipeline_grouped")


def vit_check_status(h, stream=0) -> None:
    _check(lib().vit_check_status(h, stream), "vit_check_status")


def vit_debug_wait_probe(h, limit_cycles, stream=0) -> None:
    _check(lib().vit_debug_wait_probe(h, int(limit_cycles), stream), "vit_debug_wait_probe")


def vit_launch_count(h) -> int:
    return lib().vit_launch_count(h)


def vit_profile_enable(h, on: bool) -> None:
    _check(lib().vit_profile_enable(h, 1 if on else 0), "vit_profile_enable")


def vit_profile_collect(h) -> dict:
    """{class name: (milliseconds, launches)} since profiling was enabled or last collected."""
    n = len(PROF_CLASSES)
    ms = (ctypes.c_double * n)()
    cnt = (c_uint64 * n)()
    _check(lib().vit_profile_collect(h, ms, cnt), "vit_profile_collect")
    return {PROF_CLASSES[i]: (ms[i], int(cnt[i])) for i in range(n)}


def _partition_call(layer_time, out_bytes, layer_mem, device_mem, bandwidth, category_count=None):
    lt = np.ascontiguousarray(layer_time, dtype=np.float64)
    D, Lr = lt.shape
    ob = np.ascontiguousarray(out_bytes, dtype=np.float64)
    lm = np.ascontiguousarray(layer_mem, dtype=np.float64)
    dm = np.ascontiguousarray(device_mem, dtype=np.float64)
    bw = np.ascontiguousarray(bandwidth, dtype=np.float64)
    if ob.shape != (Lr,) or lm.shape != (Lr,) or dm.shape != (D,) or bw.shape != (D, D):
        raise ValueError("inconsistent partition problem shapes")
    prob = VitPartitionProblem(Lr, D, lt.ctypes.data, ob.ctypes.data, lm.ctypes.data, dm.ctypes.data, bw.ctypes.data)
    total = D if category_count is None else int(np.sum(category_count))
    n = max(1, min(Lr, total))
    layers = np.zeros(n, dtype=np.int32)
    devs = np.zeros(n, dtype=np.int32)
    t = ctypes.c_double()
    ns = c_int32()
    if category_count is None:
        st = lib().vit_partition(byref(prob), byref(t), byref(ns), layers.ctypes.data, devs.ctypes.data)
        _check(st, "vit_partition")
    else:
        cc = np.ascontiguousarray(category_count, dtype=np.int32)
        if cc.shape != (D,):
            raise ValueError("one count per category")
        st = lib().vit_partition_categories(byref(prob), cc.ctypes.data, byref(t), byref(ns), layers.ctypes.data,
                                            devs.ctypes.data)
        _check(st, "vit_partition_categories")
    k = ns.value
    return t.value, [(int(layers[i]), int(devs[i])) for i in range(k)]


def vit_partition(layer_time, out_bytes, layer_mem, device_mem, bandwidth):
    """Host-side pipeline partitioner.  Returns (T_opt, [(layer_count, device), ...])."""
    return _partition_call(layer_time, out_bytes, layer_mem, device_mem, bandwidth)


def vit_partition_categories(layer_time, out_bytes, layer_mem, device_mem, bandwidth, category_count):
    """The same with identical devices grouped; devices in the result are category indices."""
    return _partition_call(layer_time, out_bytes, layer_mem, device_mem, bandwidth, category_count)


def vit_op_layernorm(h, dtype, rows, cols, x, gain, shift, eps, y, stream=0):
    _check(lib().vit_op_layernorm(h, dtype, rows, cols, x, gain, shift, eps, y, stream), "vit_op_layernorm")


def vit_op_linear(h, dtype, M, N, K, a, w, bias, epilogue, residual, out, stream=0):
    _check(lib().vit_op_linear(h, dtype, M, N, K, a, w, bias, epilogue, residual, out, stream), "vit_op_linear")


def vit_op_linear_tiled(h, dtype, M, N, K, a, w, bias, epilogue, residual, out, tiling, stream=0):
    _check(lib().vit_op_linear_tiled(h, dtype, M, N, K, a, w, bias, epilogue, residual, out, tiling, stream),
           "vit_op_linear_tiled")


def vit_op_rowstats(h, rows, cols, x, eps, stats, stream=0):
    _check(lib().vit_op_rowstats(h, rows, cols, x, eps, stats, stream), "vit_op_rowstats")


def vit_op_linear_ln(h, M, N, K, a, stats, wg, c1, c0, gelu, out, tiling=0, stream=0):
    _check(lib().vit_op_linear_ln(h, M, N, K, a, stats, wg, c1, c0, 1 if gelu else 0, out, tiling, stream),
           "vit_op_linear_ln")


def vit_op_attention(h, dtype, images, T, heads, d, qkv, out, stream=0):
    _check(lib().vit_op_attention(h, dtype, images, T, heads, d, qkv, out, stream), "vit_op_attention")


# ---- convenience object: owns a handle and torch-allocated buffers --------------------------------
class VitModel:
    """A model instance plus torch-allocated workspaces.  All compute happens in the library."""

    def __init__(self, shape, host_params: np.ndarray, dtype=VIT_BF16, max_microbatch=1, device="cuda:0"):
        import torch
        self.torch = torch
        self.shape = shape
        self.device = torch.device(device)
        self.cfg = make_config(shape, dtype, max_microbatch)
        self.act_dtype = torch.bfloat16 if dtype == VIT_BF16 else torch.float32
        self.T = (shape.image_size // shape.patch_size) ** 2 + 1 + int(getattr(shape, "extra_tokens", 0))
        with torch.cuda.device(self.device):
            self.h = vit_create(self.cfg, host_params)
        self._ws = {}

    def close(self):
        if getattr(self, "h", None):
            with self.torch.cuda.device(self.device):
                vit_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _stream(self, stream):
        return (stream or self.torch.cuda.current_stream(self.device)).cuda_stream

    def workspace(self, microbatch, key="default"):
        n = vit_workspace_bytes(self.cfg, microbatch)
        buf = self._ws.get(key)
        if buf is None or buf.numel() < n:
            buf = self.torch.empty(n, dtype=self.torch.uint8, device=self.device)
            self._ws[key] = buf
        return buf

    def patch_embed(self, pixels, stream=None):
        mb = pixels.shape[0]
        assert pixels.dtype == self.torch.float32 and pixels.is_contiguous()
        out = self.torch.empty((mb, self.T, self.shape.hidden), dtype=self.act_dtype, device=self.device)
        ws = self.workspace(mb)
        vit_patch_embed(self.h, mb, pixels.data_ptr(), out.data_ptr(), ws.data_ptr(), ws.numel(), self._stream(stream))
        return out

    def run_stage(self, layer_begin, layer_end, x, out=None, stream=None):
        mb = x.shape[0]
        assert x.dtype == self.act_dtype and x.is_contiguous()
        if out is None:
            out = self.torch.empty_like(x)
        ws = self.workspace(mb)
        vit_run_stage(self.h, layer_begin, layer_end, mb, x.data_ptr(), out.data_ptr(), ws.data_ptr(),
                      ws.numel(), self._stream(stream))
        return out

    def head(self, x, stream=None):
        mb = x.shape[0]
        logits = self.torch.empty((mb, self.shape.num_classes), dtype=self.torch.float32, device=self.device)
        ws = self.workspace(mb)
        vit_head(self.h, mb, x.data_ptr(), logits.data_ptr(), ws.data_ptr(), ws.numel(), self._stream(stream))
        return logits

    def forward(self, pixels, stages=None):
        stages = stages or [(0, self.shape.layers)]
        x = self.patch_embed(pixels)
        for lb, le in stages:
            x = self.run_stage(lb, le, x, out=x)
        return self.head(x)

    def make_pipeline_buffers(self, microbatch, n_streams):
        n = vit_pipeline_workspace_bytes(self.cfg, microbatch)
        wss = [self.torch.empty(n, dtype=self.torch.uint8, device=self.device) for _ in range(n_streams)]
        streams = [self.torch.cuda.Stream(self.device) for _ in range(n_streams)]
        return wss, streams, n

    def run_pipeline(self, stage_layers, microbatch, pixels, logits, wss, streams, ws_bytes, host=False, group=1):
        batch = pixels.shape[0]
        if group > 1:
            vit_run_pipeline_grouped(self.h, list(stage_layers), batch, microbatch, group, pixels.data_ptr(),
                                     logits.data_ptr(), [w.data_ptr() for w in wss], ws_bytes,
                                     [s.cuda_stream for s in streams])
            return
        fn = vit_run_pipeline_host if host else vit_run_pipeline
        fn(self.h, list(stage_layers), batch, microbatch, pixels.data_ptr(), logits.data_ptr(),
           [w.data_ptr() for w in wss], ws_bytes, [s.cuda_stream for s in streams])

    def check(self, stream=None):
        vit_check_status(self.h, self._stream(stream))

    @property
    def launches(self):
        return vit_launch_count(self.h)

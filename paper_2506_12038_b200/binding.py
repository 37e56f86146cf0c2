"""Thin ctypes binding of the C ABI in include/lcd.h: argument marshalling only.

Every step of the path (index packing, input transformation, table lookup and accumulation) runs inside
liblcd_b200.so; torch is used for device memory and streams.  There is no CPU fallback: if the shared
library is missing, importing this module raises.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import c_char_p, c_int, c_int64, c_size_t, c_void_p, POINTER, Structure, byref

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liblcd_b200.so")

LCD_OK = 0
STATUS_NAMES = {0: "LCD_OK", 1: "LCD_ERR_INVALID_ARG", 2: "LCD_ERR_UNSUPPORTED", 3: "LCD_ERR_BUFFER_TOO_SMALL",
                4: "LCD_ERR_INDEX_RANGE", 5: "LCD_ERR_BAD_BLOB", 6: "LCD_ERR_CUDA", 7: "LCD_ERR_TIMEOUT"}
ALGO_AUTO, ALGO_REFERENCE, ALGO_BUCKET_LUT, ALGO_REGISTER_LUT, ALGO_DENSE_TC, ALGO_DENSE_F16, ALGO_TC_LUT = 0, 1, 2, 3, 4, 5, 6
ALGO_SHARED_BUCKET = 7
HEADER_BYTES = 64
MAX_BATCH = 8

EXPORTS = ["lcd_status_string", "lcd_last_cuda_error", "lcd_packed_weights_bytes", "lcd_pack_weights",
           "lcd_unpack_weights", "lcd_smooth_quantize_act", "lcd_lut_linear_workspace_bytes", "lcd_lut_linear",
           "lcd_linear_host_scratch_bytes", "lcd_linear_host", "lcd_smooth_quantize_act_batch",
           "lcd_lut_linear_batch_workspace_bytes", "lcd_lut_linear_batch", "lcd_lut_linear_batch_resolve", "lcd_lut_linear_static",
           "lcd_linear_host_batch_sizes", "lcd_linear_host_batch", "lcd_lut_linear_act8",
           "lcd_lut_linear_batch_act8", "lcd_linear_fused_batch_workspace_bytes", "lcd_linear_fused_batch",
           "lcd_smoothing_search_workspace_bytes", "lcd_smoothing_search", "lcd_reclassify",
           "lcd_dbci_workspace_bytes", "lcd_dbci"]
STATIC_SCRATCH_BYTES = 4 << 20


class DbciResult(Structure):
    """lcd_dbci_result"""
    _fields_ = [("sigma", ctypes.c_double), ("eps", ctypes.c_double), ("min_pts", c_int64), ("left", c_int64),
                ("right", c_int64), ("n_centroids", ctypes.c_int32), ("n_noise", ctypes.c_int32),
                ("n_clusters_found", ctypes.c_int32)]


class FusedProblem(Structure):
    """lcd_fused_problem"""
    _fields_ = [("packed_weights_dev", c_void_p), ("header_host", c_void_p), ("x_fp16", c_void_p), ("M", c_int64),
                ("ldx", c_int64), ("inv_smooth", c_void_p), ("y", c_void_p), ("ldy", c_int64)]


class ActProblem(Structure):
    """lcd_act_problem"""
    _fields_ = [("x_fp16", c_void_p), ("M", c_int64), ("K", c_int64), ("ldx", c_int64), ("inv_smooth", c_void_p),
                ("static_scale", c_void_p), ("act_idx", c_void_p), ("act_scale", c_void_p)]


class HostProblem(Structure):
    """lcd_host_problem"""
    _fields_ = [("packed_weights_dev", c_void_p), ("header_host", c_void_p), ("inv_smooth", c_void_p), ("M", c_int64)]


class LinearProblem(Structure):
    """lcd_linear_problem"""
    _fields_ = [("packed_weights_dev", c_void_p), ("header_host", c_void_p), ("act_idx", c_void_p),
                ("act_scale", c_void_p), ("M", c_int64), ("y", c_void_p), ("ldy", c_int64)]


class LcdError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str = ""):
        self.status = status
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)} {detail}".strip())


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} not built: run `python paper_2506_12038_b200/build.py` "
                          "(there is no fallback path)")
    lib = ctypes.CDLL(LIB_PATH)
    lib.lcd_status_string.restype = c_char_p
    lib.lcd_status_string.argtypes = [c_int]
    lib.lcd_last_cuda_error.restype = c_char_p
    lib.lcd_packed_weights_bytes.argtypes = [c_int64, c_int64, c_int, POINTER(c_size_t)]
    lib.lcd_pack_weights.argtypes = [c_void_p, c_void_p, c_int64, c_int64, c_int, c_int, c_void_p, c_size_t,
                                     POINTER(c_int64), POINTER(c_int64)]
    lib.lcd_unpack_weights.argtypes = [c_void_p, c_size_t, c_void_p, c_void_p, POINTER(c_int64), POINTER(c_int64),
                                       POINTER(c_int), POINTER(c_int)]
    lib.lcd_smooth_quantize_act.argtypes = [c_void_p, c_int64, c_int64, c_int64, c_void_p, c_void_p, c_int,
                                            c_void_p, c_void_p, c_void_p]
    lib.lcd_lut_linear_workspace_bytes.argtypes = [c_void_p, c_int64, c_int, POINTER(c_size_t)]
    lib.lcd_lut_linear.argtypes = [c_void_p, c_void_p, c_void_p, c_void_p, c_int64, c_void_p, c_int64, c_int,
                                   c_void_p, c_size_t, c_void_p, c_void_p]
    lib.lcd_lut_linear_act8.argtypes = lib.lcd_lut_linear.argtypes
    lib.lcd_dbci_workspace_bytes.argtypes = [c_int64, c_int, POINTER(c_size_t)]
    lib.lcd_dbci.argtypes = [c_void_p, c_int64, c_void_p, c_size_t, c_void_p, c_int, c_void_p, c_void_p, c_void_p, c_void_p]
    lib.lcd_reclassify.argtypes = [c_void_p, c_void_p, c_void_p, c_int64, c_int64, c_int64, c_int, c_void_p, c_void_p,
                                   c_void_p, c_void_p]
    lib.lcd_smoothing_search_workspace_bytes.argtypes = [c_int64, c_int64, c_int, POINTER(c_size_t)]
    lib.lcd_smoothing_search.argtypes = [c_void_p, c_int64, c_int64, c_int64, c_void_p, c_void_p, c_int, c_void_p, c_size_t,
                                         c_void_p, c_void_p, c_void_p, c_void_p]
    lib.lcd_linear_fused_batch_workspace_bytes.argtypes = [POINTER(FusedProblem), c_int, c_int, POINTER(c_size_t)]
    lib.lcd_linear_fused_batch.argtypes = [POINTER(FusedProblem), c_int, c_int, c_void_p, c_size_t, c_void_p, c_void_p]
    lib.lcd_lut_linear_batch_act8.argtypes = [POINTER(LinearProblem), c_int, c_int, c_void_p, c_size_t, c_void_p, c_void_p]
    lib.lcd_linear_host_scratch_bytes.argtypes = [c_void_p, c_int64, POINTER(c_size_t)]
    lib.lcd_linear_host.argtypes = [c_void_p, c_void_p, c_void_p, c_int64, c_void_p, c_void_p, c_void_p, c_size_t,
                                    c_void_p, c_void_p]
    lib.lcd_smooth_quantize_act_batch.argtypes = [POINTER(ActProblem), c_int, c_int, c_void_p]
    lib.lcd_lut_linear_batch_workspace_bytes.argtypes = [POINTER(LinearProblem), c_int, c_int, POINTER(c_size_t)]
    lib.lcd_lut_linear_batch.argtypes = [POINTER(LinearProblem), c_int, c_int, c_void_p, c_size_t, c_void_p, c_void_p]
    lib.lcd_lut_linear_batch_resolve.argtypes = [POINTER(LinearProblem), c_int, c_int, POINTER(c_int)]
    lib.lcd_lut_linear_static.argtypes = [c_void_p, c_void_p, c_void_p, c_void_p, c_int64, c_void_p, c_int64, c_int,
                                          c_void_p, c_void_p]
    lib.lcd_linear_host_batch_sizes.argtypes = [POINTER(HostProblem), c_int, POINTER(c_size_t), POINTER(c_size_t),
                                                POINTER(c_size_t)]
    lib.lcd_linear_host_batch.argtypes = [POINTER(HostProblem), c_int, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p,
                                          c_void_p]
    for name in EXPORTS:
        if name not in ("lcd_status_string", "lcd_last_cuda_error"):
            getattr(lib, name).restype = c_int
    return lib


lib = _load()


def _check(st: int, where: str):
    if st != LCD_OK:
        detail = lib.lcd_last_cuda_error().decode() if st == 6 else ""
        raise LcdError(st, where, detail)


def _np_ptr(a: np.ndarray) -> c_void_p:
    return c_void_p(a.ctypes.data)


# ------------------------------------------------------------------------------------------- host: packing
def packed_weights_bytes(N: int, K: int, bits: int) -> int:
    out = c_size_t(0)
    _check(lib.lcd_packed_weights_bytes(N, K, bits, byref(out)), "lcd_packed_weights_bytes")
    return out.value


def pack_weights(idx: np.ndarray, codebook_fp16: np.ndarray, bits: int, C: int | None = None) -> np.ndarray:
    """idx uint8 [N,K], codebook fp16 [N,C] (host numpy) -> blob (host numpy uint8)."""
    idx = np.ascontiguousarray(idx, dtype=np.uint8)
    N, K = idx.shape
    C = (1 << bits) if C is None else C
    cb = np.ascontiguousarray(codebook_fp16, dtype=np.float16)
    if cb.shape != (N, C):
        raise ValueError("codebook shape")
    size = packed_weights_bytes(N, K, bits)
    out = np.empty(size, dtype=np.uint8)
    bn, bk = c_int64(-1), c_int64(-1)
    st = lib.lcd_pack_weights(_np_ptr(idx), _np_ptr(cb), N, K, bits, C, _np_ptr(out), size, byref(bn), byref(bk))
    if st == 4:
        raise LcdError(st, "lcd_pack_weights", f"at n={bn.value} k={bk.value}")
    _check(st, "lcd_pack_weights")
    return out


def unpack_weights(blob: np.ndarray):
    blob = np.ascontiguousarray(blob, dtype=np.uint8)
    N, K, bits, C = c_int64(), c_int64(), c_int(), c_int()
    _check(lib.lcd_unpack_weights(_np_ptr(blob), blob.size, None, None, byref(N), byref(K), byref(bits), byref(C)),
           "lcd_unpack_weights")
    idx = np.empty((N.value, K.value), dtype=np.uint8)
    cb = np.empty((N.value, C.value), dtype=np.float16)
    _check(lib.lcd_unpack_weights(_np_ptr(blob), blob.size, _np_ptr(idx), _np_ptr(cb), byref(N), byref(K),
                                  byref(bits), byref(C)), "lcd_unpack_weights")
    return idx, cb, bits.value, C.value


# ------------------------------------------------------------------------------------------- device calls
def _stream_ptr(stream=None) -> c_void_p:
    import torch
    s = torch.cuda.current_stream() if stream is None else stream
    return c_void_p(s.cuda_stream)


class PackedWeights:
    """A blob resident on the device plus the host copy of its 64-byte header."""

    def __init__(self, blob: np.ndarray, device="cuda"):
        import torch
        self.header = bytes(blob[:HEADER_BYTES])
        self._hdr_buf = ctypes.create_string_buffer(self.header, HEADER_BYTES)
        f = np.frombuffer(self.header, dtype="<u8")
        self.N, self.K, self.K_pad = int(f[1]), int(f[2]), int(f[3])
        u = np.frombuffer(self.header, dtype="<u4")
        self.bits, self.C = int(u[8]), int(u[9])
        self.nbytes = int(blob.size)
        self.dev = torch.from_numpy(np.ascontiguousarray(blob)).to(device)
        assert self.dev.data_ptr() % 256 == 0

    @property
    def header_ptr(self) -> c_void_p:
        return ctypes.cast(self._hdr_buf, c_void_p)


def smooth_quantize_act(x, inv_smooth=None, static_scale=None, act_idx=None, act_scale=None, stream=None,
                        act_bits: int = 4):
    """x: CUDA fp16 [M,K] (row stride may exceed K) -> (act_idx uint8 [M,K_pad/2], act_scale fp32 [M]); with
    act_bits = 8 the levels come back as int8 [M,K_pad]."""
    import torch
    assert x.is_cuda and x.dtype == torch.float16 and x.dim() == 2 and x.stride(1) == 1
    M, K = x.shape
    K_pad = (K + 255) // 256 * 256
    assert act_bits in (4, 8)
    if act_idx is None:
        act_idx = (torch.empty((M, K_pad // 2), dtype=torch.uint8, device=x.device) if act_bits == 4 else
                   torch.empty((M, K_pad), dtype=torch.int8, device=x.device))
    assert act_idx.dtype == (torch.uint8 if act_bits == 4 else torch.int8)
    if act_scale is None:
        act_scale = torch.empty((M,), dtype=torch.float32, device=x.device)
    st = lib.lcd_smooth_quantize_act(c_void_p(x.data_ptr()), M, K, x.stride(0),
                                     c_void_p(inv_smooth.data_ptr()) if inv_smooth is not None else None,
                                     c_void_p(static_scale.data_ptr()) if static_scale is not None else None,
                                     act_bits, c_void_p(act_idx.data_ptr()), c_void_p(act_scale.data_ptr()),
                                     _stream_ptr(stream))
    _check(st, "lcd_smooth_quantize_act")
    return act_idx, act_scale


def lut_linear_workspace_bytes(w: PackedWeights, M: int, algo: int = ALGO_AUTO) -> int:
    out = c_size_t(0)
    _check(lib.lcd_lut_linear_workspace_bytes(w.header_ptr, M, algo, byref(out)), "lcd_lut_linear_workspace_bytes")
    return out.value


def lut_linear(w: PackedWeights, act_idx, act_scale, y=None, algo: int = ALGO_AUTO, workspace=None,
               status_word=None, stream=None):
    """y[m][n] = s_q[m] * sum_k q[m][k] * cb[n][idx[n][k]]  (CUDA fp32 [M,N]).  act_idx: uint8 packed 4-bit
    levels, or int8 8-bit levels (as smooth_quantize_act returns them for act_bits = 8)."""
    import torch
    M = act_idx.shape[0]
    fn, name = ((lib.lcd_lut_linear_act8, "lcd_lut_linear_act8") if act_idx.dtype == torch.int8 else
                (lib.lcd_lut_linear, "lcd_lut_linear"))
    if y is None:
        y = torch.empty((M, w.N), dtype=torch.float32, device=act_idx.device)
    need = lut_linear_workspace_bytes(w, M, algo)
    if need and (workspace is None or workspace.numel() * workspace.element_size() < need):
        workspace = torch.zeros(need, dtype=torch.uint8, device=act_idx.device)   # must start zero-filled
    st = fn(c_void_p(w.dev.data_ptr()), w.header_ptr, c_void_p(act_idx.data_ptr()),
                            c_void_p(act_scale.data_ptr()), M, c_void_p(y.data_ptr()), y.stride(0), algo,
                            c_void_p(workspace.data_ptr()) if workspace is not None else None,
                            workspace.numel() * workspace.element_size() if workspace is not None else 0,
                            c_void_p(status_word.data_ptr()) if status_word is not None else None,
                            _stream_ptr(stream))
    _check(st, name)
    return y


def lut_linear_static(w: PackedWeights, act_idx, act_scale, y, algo: int = ALGO_AUTO, status_word=None, stream=None):
    """lcd_lut_linear_static: M <= 16 lookup whose scratch is the library's built-in device array.  Nothing is
    allocated here either: the caller passes y (CUDA fp32 [M, >= N]).  Calls must not overlap on the GPU."""
    M = act_idx.shape[0]
    st = lib.lcd_lut_linear_static(c_void_p(w.dev.data_ptr()), w.header_ptr, c_void_p(act_idx.data_ptr()),
                                   c_void_p(act_scale.data_ptr()), M, c_void_p(y.data_ptr()), y.stride(0), algo,
                                   c_void_p(status_word.data_ptr()) if status_word is not None else None,
                                   _stream_ptr(stream))
    _check(st, "lcd_lut_linear_static")
    return y


class ActBatch:
    """Up to MAX_BATCH activation matrices quantised by one launch.  items: (x, inv_smooth, act_idx, act_scale)
    CUDA tensors (inv_smooth may be None); the argument array is built once and reused by run().  The level
    width follows the dtype of the act_idx tensors: uint8 = packed 4-bit, int8 = 8-bit."""

    def __init__(self, items):
        import torch
        self._keep = list(items)
        self.act_bits = 8 if self._keep[0][2].dtype == torch.int8 else 4
        assert all((it[2].dtype == torch.int8) == (self.act_bits == 8) for it in self._keep)
        self.count = len(self._keep)
        self.arr = (ActProblem * self.count)()
        for a, (x, inv_s, idx, scale) in zip(self.arr, self._keep):
            a.x_fp16, a.M, a.K, a.ldx = x.data_ptr(), x.shape[0], x.shape[1], x.stride(0)
            a.inv_smooth = inv_s.data_ptr() if inv_s is not None else None
            a.static_scale = None
            a.act_idx, a.act_scale = idx.data_ptr(), scale.data_ptr()

    def run(self, stream=None):
        _check(lib.lcd_smooth_quantize_act_batch(self.arr, self.count, self.act_bits, _stream_ptr(stream)),
               "lcd_smooth_quantize_act_batch")


def dbci(weights, max_centroids: int = 4096, want_labels: bool = True, stream=None):
    """Section 3.1 on a flat CUDA fp32 tensor.  Returns a dict: sigma, eps, min_pts, left, right, n_noise,
    n_clusters_found, centroids (CUDA fp32, ascending), sorted (CUDA fp32) and labels (CUDA int32, in sorted order)."""
    import torch
    w = weights.reshape(-1)
    assert w.is_cuda and w.dtype == torch.float32 and w.is_contiguous()
    n = w.numel()
    need = c_size_t(0)
    _check(lib.lcd_dbci_workspace_bytes(n, max_centroids, byref(need)), "lcd_dbci_workspace_bytes")
    ws = torch.empty(need.value, dtype=torch.uint8, device=w.device)
    cents = torch.empty((max_centroids,), dtype=torch.float32, device=w.device)
    labels = torch.empty((n,), dtype=torch.int32, device=w.device) if want_labels else None
    srt = torch.empty((n,), dtype=torch.float32, device=w.device)
    res = torch.zeros((ctypes.sizeof(DbciResult),), dtype=torch.uint8, device=w.device)
    _check(lib.lcd_dbci(c_void_p(w.data_ptr()), n, c_void_p(ws.data_ptr()), need.value, c_void_p(cents.data_ptr()),
                        max_centroids, c_void_p(labels.data_ptr()) if labels is not None else None,
                        c_void_p(srt.data_ptr()), c_void_p(res.data_ptr()), _stream_ptr(stream)), "lcd_dbci")
    r = DbciResult.from_buffer_copy(res.cpu().numpy().tobytes())
    return {"sigma": r.sigma, "eps": r.eps, "min_pts": r.min_pts, "left": r.left, "right": r.right,
            "n_noise": r.n_noise, "n_clusters_found": r.n_clusters_found,
            "centroids": cents[:min(r.n_centroids, max_centroids)], "sorted": srt, "labels": labels}


def reclassify(idx, codebook, delta_w, stream=None, out=None):
    """Section 3.2 bookkeeping.  idx: CUDA uint8 [N,K]; codebook: CUDA fp16 [N,C] rows ascending; delta_w: CUDA fp32
    [N,K].  Returns (new_idx uint8 [N,K], delta_c fp64 [N,C], counts int32 [N,C]); `out` may give those three
    tensors to write into."""
    import torch
    assert idx.dtype == torch.uint8 and codebook.dtype == torch.float16 and delta_w.dtype == torch.float32
    assert idx.is_contiguous() and codebook.is_contiguous() and delta_w.stride(1) == 1
    N, K = idx.shape
    C = codebook.shape[1]
    if out is None:
        new_idx = torch.empty_like(idx)
        delta_c = torch.empty((N, C), dtype=torch.float64, device=idx.device)
        counts = torch.empty((N, C), dtype=torch.int32, device=idx.device)
    else:
        new_idx, delta_c, counts = out
        assert new_idx.dtype == torch.uint8 and delta_c.dtype == torch.float64 and counts.dtype == torch.int32
        assert new_idx.shape == idx.shape and delta_c.shape == (N, C) and counts.shape == (N, C)
    _check(lib.lcd_reclassify(c_void_p(idx.data_ptr()), c_void_p(codebook.data_ptr()), c_void_p(delta_w.data_ptr()), N, K,
                              delta_w.stride(0), C, c_void_p(new_idx.data_ptr()), c_void_p(delta_c.data_ptr()),
                              c_void_p(counts.data_ptr()), _stream_ptr(stream)), "lcd_reclassify")
    return new_idx, delta_c, counts


def smoothing_search(x, wmax, alphas, stream=None):
    """Section 3.4 grid search on a calibration batch.  x: CUDA fp16 [T,K]; wmax: CUDA fp32 [K]; alphas: list of
    floats.  Returns (best index tensor int32 [1], mse fp64 [G], inv_smooth fp32 [K]) on the device."""
    import torch
    assert x.is_cuda and x.dtype == torch.float16 and x.dim() == 2 and x.stride(1) == 1
    T, K = x.shape
    G = len(alphas)
    need = c_size_t(0)
    _check(lib.lcd_smoothing_search_workspace_bytes(T, K, G, byref(need)), "lcd_smoothing_search_workspace_bytes")
    ws = torch.empty(need.value, dtype=torch.uint8, device=x.device)
    mse = torch.empty((G,), dtype=torch.float64, device=x.device)
    best = torch.empty((1,), dtype=torch.int32, device=x.device)
    inv = torch.empty((K,), dtype=torch.float32, device=x.device)
    al = (ctypes.c_float * G)(*[float(a) for a in alphas])
    _check(lib.lcd_smoothing_search(c_void_p(x.data_ptr()), T, K, x.stride(0), c_void_p(wmax.data_ptr()), al, G,
                                    c_void_p(ws.data_ptr()), need.value, c_void_p(mse.data_ptr()),
                                    c_void_p(best.data_ptr()), c_void_p(inv.data_ptr()), _stream_ptr(stream)),
           "lcd_smoothing_search")
    return best, mse, inv


def resolve_batch_algo(weights_and_tokens, algo: int = ALGO_AUTO) -> int:
    """The kernel family a grouped (or fused) call over these (PackedWeights, M) pairs runs for `algo`."""
    items = list(weights_and_tokens)
    arr = (LinearProblem * len(items))()
    for a, (w, M) in zip(arr, items):
        a.header_host, a.M = w.header_ptr, M
    out = c_int(0)
    _check(lib.lcd_lut_linear_batch_resolve(arr, len(items), algo, byref(out)), "lcd_lut_linear_batch_resolve")
    return out.value


class FusedBatch:
    """Up to MAX_BATCH independent problems from x to y in one call: items are (PackedWeights, x fp16 [M,K] CUDA,
    inv_smooth or None, y fp32 [M,N] CUDA).  Every M <= 16: ONE launch that quantises the activations and runs the
    lookup.  Every M > 16: one launch that quantises all inputs, then the tensor-core kernel per problem."""

    def __init__(self, items, algo: int = ALGO_AUTO, status_word=None):
        import torch
        self._keep = list(items)
        self.count = len(self._keep)
        self.algo = algo
        self.arr = (FusedProblem * self.count)()
        for a, (w, x, inv_s, y) in zip(self.arr, self._keep):
            assert x.dtype == torch.float16 and x.stride(1) == 1 and y.dtype == torch.float32
            a.packed_weights_dev, a.header_host = w.dev.data_ptr(), w.header_ptr
            a.x_fp16, a.M, a.ldx = x.data_ptr(), x.shape[0], x.stride(0)
            a.inv_smooth = inv_s.data_ptr() if inv_s is not None else None
            a.y, a.ldy = y.data_ptr(), y.stride(0)
        need = c_size_t(0)
        _check(lib.lcd_linear_fused_batch_workspace_bytes(self.arr, self.count, algo, byref(need)),
               "lcd_linear_fused_batch_workspace_bytes")
        self.workspace = torch.zeros(max(need.value, 256), dtype=torch.uint8, device=self._keep[0][1].device)
        self.status_word = status_word

    def run(self, stream=None):
        _check(lib.lcd_linear_fused_batch(self.arr, self.count, self.algo, c_void_p(self.workspace.data_ptr()),
                                          self.workspace.numel(),
                                          c_void_p(self.status_word.data_ptr()) if self.status_word is not None else None,
                                          _stream_ptr(stream)), "lcd_linear_fused_batch")


class LinearBatch:
    """Up to MAX_BATCH independent lookup problems (M <= 16, same index width) run by one launch.
    items: (PackedWeights, act_idx, act_scale, y) with CUDA tensors; the zero-filled workspace is owned here.
    act_idx tensors of dtype int8 are 8-bit levels (all items alike)."""

    def __init__(self, items, algo: int = ALGO_AUTO, status_word=None):
        import torch
        self._keep = list(items)
        self.act8 = self._keep[0][1].dtype == torch.int8
        assert all((it[1].dtype == torch.int8) == self.act8 for it in self._keep)
        self.count = len(self._keep)
        self.algo = algo
        self.arr = (LinearProblem * self.count)()
        for a, (w, idx, scale, y) in zip(self.arr, self._keep):
            a.packed_weights_dev, a.header_host = w.dev.data_ptr(), w.header_ptr
            a.act_idx, a.act_scale, a.M = idx.data_ptr(), scale.data_ptr(), idx.shape[0]
            a.y, a.ldy = y.data_ptr(), y.stride(0)
        need = c_size_t(0)
        _check(lib.lcd_lut_linear_batch_workspace_bytes(self.arr, self.count, algo, byref(need)),
               "lcd_lut_linear_batch_workspace_bytes")
        self.workspace = torch.zeros(max(need.value, 256), dtype=torch.uint8, device=self._keep[0][1].device)
        self.status_word = status_word

    def run(self, stream=None):
        fn = lib.lcd_lut_linear_batch_act8 if self.act8 else lib.lcd_lut_linear_batch
        _check(fn(self.arr, self.count, self.algo, c_void_p(self.workspace.data_ptr()), self.workspace.numel(),
                  c_void_p(self.status_word.data_ptr()) if self.status_word is not None else None,
                  _stream_ptr(stream)), "lcd_lut_linear_batch")


class HostBatch:
    """lcd_linear_host_batch: up to MAX_BATCH problems (M <= 16) from pinned host inputs to pinned host outputs with
    one copy in and one copy out.  items: (PackedWeights, inv_smooth CUDA tensor or None, M).  The pinned staging
    tensors x_host (uint8) / y_host (uint8) and the device scratch are owned here; x_view(i) / y_view(i) give
    problem i's fp16 [M, K] input and fp32 [M, N] output inside them."""

    def __init__(self, items, device="cuda", status_word=None):
        import torch
        self._keep = list(items)
        self.status_word = status_word
        self.count = len(self._keep)
        self.arr = (HostProblem * self.count)()
        for a, (w, inv_s, M) in zip(self.arr, self._keep):
            a.packed_weights_dev, a.header_host = w.dev.data_ptr(), w.header_ptr
            a.inv_smooth = inv_s.data_ptr() if inv_s is not None else None
            a.M = M
        xb, yb, sb = c_size_t(0), c_size_t(0), c_size_t(0)
        _check(lib.lcd_linear_host_batch_sizes(self.arr, self.count, byref(xb), byref(yb), byref(sb)),
               "lcd_linear_host_batch_sizes")
        self.x_host = torch.zeros(xb.value, dtype=torch.uint8).pin_memory()
        self.y_host = torch.zeros(yb.value, dtype=torch.uint8).pin_memory()
        self.scratch = torch.zeros(sb.value, dtype=torch.uint8, device=device)     # zero-filled once, kept usable by the calls
        self._x_off, self._y_off, xo, yo = [], [], 0, 0
        for w, _, M in self._keep:
            self._x_off.append(xo)
            self._y_off.append(yo)
            xo += (M * w.K * 2 + 15) // 16 * 16
            yo += (M * w.N * 4 + 15) // 16 * 16

    def x_view(self, i):
        import torch
        w, _, M = self._keep[i]
        return self.x_host[self._x_off[i]:self._x_off[i] + M * w.K * 2].view(torch.float16).view(M, w.K)

    def y_view(self, i):
        import torch
        w, _, M = self._keep[i]
        return self.y_host[self._y_off[i]:self._y_off[i] + M * w.N * 4].view(torch.float32).view(M, w.N)

    def capture(self):
        """Records one call (copy in, launches, copy out) as a CUDA graph; run() without a stream replays it
        from then on: one graph launch instead of two copies and the kernel launches.  The buffers are owned
        here and keep their addresses, so the recording stays valid."""
        import torch
        self.run()                                   # first-use set-up (function attributes) outside the capture
        torch.cuda.current_stream().synchronize()
        side = torch.cuda.Stream(device=self.scratch.device)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                self._enqueue(None)
        self._graph = graph
        return self

    def run(self, stream=None):
        if stream is None and getattr(self, "_graph", None) is not None:
            self._graph.replay()
            return
        self._enqueue(stream)

    def _enqueue(self, stream):
        _check(lib.lcd_linear_host_batch(self.arr, self.count, c_void_p(self.x_host.data_ptr()),
                                         c_void_p(self.y_host.data_ptr()), c_void_p(self.scratch.data_ptr()),
                                         self.scratch.numel(),
                                         c_void_p(self.status_word.data_ptr()) if self.status_word is not None else None,
                                         _stream_ptr(stream)), "lcd_linear_host_batch")


def linear_host_scratch_bytes(w: PackedWeights, M: int) -> int:
    out = c_size_t(0)
    _check(lib.lcd_linear_host_scratch_bytes(w.header_ptr, M, byref(out)), "lcd_linear_host_scratch_bytes")
    return out.value


def linear_host(w: PackedWeights, x_host, inv_smooth, y_host, scratch, stream=None, status_word=None):
    """x_host: pinned CPU fp16 [M,K]; y_host: pinned CPU fp32 [M,N]; scratch: CUDA uint8, zero-filled before its first
    use; enqueues copies + kernels, no sync."""
    M = x_host.shape[0]
    st = lib.lcd_linear_host(c_void_p(w.dev.data_ptr()), w.header_ptr, c_void_p(x_host.data_ptr()), M,
                             c_void_p(inv_smooth.data_ptr()) if inv_smooth is not None else None,
                             c_void_p(y_host.data_ptr()), c_void_p(scratch.data_ptr()),
                             scratch.numel() * scratch.element_size(),
                             c_void_p(status_word.data_ptr()) if status_word is not None else None, _stream_ptr(stream))
    _check(st, "lcd_linear_host")
    return y_host

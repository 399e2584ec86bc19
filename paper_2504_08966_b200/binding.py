"""ctypes binding of libpact.so: argument marshalling only, every step runs in the CUDA kernels.

Function names follow include/pact.h.  Tensors are torch CUDA tensors; the binding passes their
data pointers and the current stream.  There is no fallback: if the library is missing or the
device is not a B200-class GPU the calls raise.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpact.so")

PACT_BF16, PACT_F32 = 0, 1
N_COUNTERS = 16
CNT = {"n_out": 0, "q": 1, "C": 2, "r": 3, "discarded": 4, "sweeps": 5, "band_dc": 6,
       "band_adc": 7, "status": 8, "m": 9}
FLAG_CENTER_ONLY, FLAG_NO_NORM, FLAG_NORM_ONLY = 1, 2, 4

EXPORTS = ["pact_create", "pact_destroy", "pact_workspace_bytes", "pact_status_string",
           "pact_last_cuda_error", "pact_importance", "pact_prune", "pact_dbdpc",
           "pact_prune_static", "pact_reincorporate", "pact_merge", "pact_reduce", "pact_reduce_host",
           "pact_host_staging_bytes", "pact_launch_count", "pact_profile_enable", "pact_profile_read",
           "pact_profile_stage_name", "pact_graph_create", "pact_graph_launch", "pact_graph_destroy",
           "pact_key_spread", "pact_set_wait_limits"]


class Params(C.Structure):
    _fields_ = [("lam", C.c_double), ("d_c", C.c_float), ("d_n", C.c_float), ("alpha", C.c_float),
                ("n_prune", C.c_int32), ("flags", C.c_uint32)]


class ImageDesc(C.Structure):
    _fields_ = [("H", C.c_void_p), ("ldH", C.c_int64), ("K_euti", C.c_void_p), ("ldKe", C.c_int64),
                ("Q_euti", C.c_void_p), ("ldQ", C.c_int64), ("K_clu", C.c_void_p), ("ldKc", C.c_int64),
                ("P", C.c_void_p), ("n_total", C.c_int32), ("vis_start", C.c_int32), ("N", C.c_int32),
                ("reserved", C.c_int32), ("H_out", C.c_void_p), ("ldHo", C.c_int64),
                ("P_out", C.c_void_p), ("size_out", C.c_void_p), ("label", C.c_void_p),
                ("score", C.c_void_p), ("keep", C.c_void_p), ("counters", C.c_void_p),
                ("logw_out", C.c_void_p)]


_lib = None


def lib():
    """Loads libpact.so (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2504_08966_b200.build`")
        L = C.CDLL(LIB_PATH)
        vp, i32, i64, sz = C.c_void_p, C.c_int, C.c_int64, C.c_size_t
        L.pact_create.argtypes = [C.POINTER(vp), i32, i32, i32, i32, i32, i32]
        L.pact_destroy.argtypes = [vp]
        L.pact_workspace_bytes.argtypes = [vp, i32, i32]
        L.pact_workspace_bytes.restype = sz
        L.pact_status_string.argtypes = [i32]
        L.pact_status_string.restype = C.c_char_p
        L.pact_last_cuda_error.argtypes = [vp]
        L.pact_last_cuda_error.restype = C.c_char_p
        L.pact_importance.argtypes = [vp, C.POINTER(ImageDesc), C.POINTER(Params), vp, vp, sz, vp]
        L.pact_prune.argtypes = [vp, vp, i32, C.POINTER(Params), vp, vp, vp, vp, vp, sz, vp]
        L.pact_prune_static.argtypes = [vp, i32, C.POINTER(Params), vp, vp, vp, vp, vp]
        L.pact_dbdpc.argtypes = [vp, vp, i64, i32, vp, vp, C.POINTER(Params), vp, vp, vp, vp, vp, vp, sz, vp]
        L.pact_reincorporate.argtypes = [vp, vp, i64, i32, vp, vp, vp, vp, C.POINTER(Params), vp, vp, vp,
                                         vp, sz, vp]
        L.pact_key_spread.argtypes = [vp, C.POINTER(vp), i32, i64, i32, C.c_float, vp, vp, vp, sz, vp]
        L.pact_merge.argtypes = [vp, C.POINTER(ImageDesc), vp, vp, vp, C.POINTER(Params), vp, sz, vp]
        L.pact_reduce.argtypes = [vp, C.POINTER(ImageDesc), i32, C.POINTER(Params), i32, vp, sz, vp]
        L.pact_reduce_host.argtypes = [vp, C.POINTER(ImageDesc), C.POINTER(Params), vp, sz, vp, sz, vp]
        L.pact_host_staging_bytes.argtypes = [vp, i32, i32]
        L.pact_host_staging_bytes.restype = sz
        L.pact_graph_create.argtypes = [vp, C.POINTER(ImageDesc), i32, C.POINTER(Params), i32, vp, sz, C.POINTER(vp)]
        L.pact_graph_launch.argtypes = [vp, vp]
        L.pact_graph_destroy.argtypes = [vp]
        L.pact_launch_count.argtypes = [vp]
        L.pact_set_wait_limits.argtypes = [vp, i32, i32]
        L.pact_launch_count.restype = C.c_longlong
        L.pact_profile_enable.argtypes = [vp, i32]
        L.pact_profile_read.argtypes = [vp, C.POINTER(C.c_float), i32]
        L.pact_profile_stage_name.argtypes = [i32]
        L.pact_profile_stage_name.restype = C.c_char_p
        for name in EXPORTS:
            if getattr(L, name).restype is C.c_int:
                getattr(L, name).restype = C.c_int
        _lib = L
    return _lib


class PactError(RuntimeError):
    pass


def _check(ctx, status: int):
    if status != 0:
        L = lib()
        msg = L.pact_status_string(status).decode()
        if status == -4 and ctx is not None:
            msg += ": " + L.pact_last_cuda_error(ctx).decode()
        raise PactError(f"pact status {status}: {msg}")


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _dt(dtype) -> int:
    if dtype == torch.bfloat16:
        return PACT_BF16
    if dtype == torch.float32:
        return PACT_F32
    raise PactError(f"unsupported dtype {dtype}")


def make_params(lam=0.5, d_c=0.3, d_n=2.0, alpha=1.5, n_prune=-1, flags=0) -> Params:
    return Params(float(lam), float(d_c), float(d_n), float(alpha), int(n_prune), int(flags))


@dataclass
class DeviceImage:
    """Device tensors of one image plus its output buffers (all owned by the caller)."""
    H: torch.Tensor
    K_euti: torch.Tensor
    Q_euti: torch.Tensor
    K_clu: torch.Tensor
    P: torch.Tensor
    vis_start: int
    N: int
    H_out: torch.Tensor
    P_out: torch.Tensor
    size_out: torch.Tensor
    label: torch.Tensor
    score: torch.Tensor
    keep: torch.Tensor
    counters: torch.Tensor
    logw_out: torch.Tensor = None

    def desc(self) -> ImageDesc:
        return ImageDesc(_ptr(self.H), self.H.stride(0), _ptr(self.K_euti), self.K_euti.stride(0),
                         _ptr(self.Q_euti), self.Q_euti.stride(0), _ptr(self.K_clu), self.K_clu.stride(0),
                         _ptr(self.P), self.H.shape[0], self.vis_start, self.N, 0,
                         _ptr(self.H_out), self.H_out.stride(0), _ptr(self.P_out), _ptr(self.size_out),
                         _ptr(self.label), _ptr(self.score), _ptr(self.keep), _ptr(self.counters),
                         _ptr(self.logw_out))


def device_image(img, out_dtype, device="cuda") -> DeviceImage:
    """Uploads a workloads.Image and allocates its outputs."""
    H = img.H.to(device)
    K = img.K.to(device)
    Kc = K if img.K_clu is None else img.K_clu.to(device)
    n_total, d = H.shape
    return DeviceImage(H, K, img.Q.to(device), Kc, img.P.to(device), img.vis_start, img.N,
                       torch.empty((n_total, d), dtype=out_dtype, device=device),
                       torch.empty(n_total, dtype=torch.int32, device=device),
                       torch.empty(n_total, dtype=torch.int32, device=device),
                       torch.empty(img.N, dtype=torch.int32, device=device),
                       torch.empty(img.N, dtype=torch.float32, device=device),
                       torch.empty(img.N, dtype=torch.uint8, device=device),
                       torch.zeros(N_COUNTERS, dtype=torch.int32, device=device),
                       torch.empty(n_total, dtype=torch.float32, device=device))


class Graph:
    """A recorded pact_reduce; launch() replays it on the current stream.  Keeps the tensors it
    points at alive."""

    def __init__(self, ctx, handle, images, ws):
        self._ctx, self.handle, self._images, self._ws = ctx, handle, images, ws

    def launch(self):
        _check(self._ctx.handle, self._ctx._L.pact_graph_launch(self.handle, _stream()))

    def close(self):
        if self.handle:
            self._ctx._L.pact_graph_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


PRUNE_STATIC_MAX_N = 65536


def pact_prune_static(score, params: Params, keep, kept_idx, pruned_idx, counts):
    """pact_prune without context or workspace, for callers that may not allocate device memory:
    the scratch is a fixed array inside the library.  score.numel() <= PRUNE_STATIC_MAX_N.
    Calls on one stream are ordered; calls that could overlap on the GPU share the array and race."""
    _check(None, lib().pact_prune_static(_ptr(score), score.numel(), C.byref(params), _ptr(keep), _ptr(kept_idx),
                                         _ptr(pruned_idx), _ptr(counts), _stream()))


class Context:
    """Owns a pact_ctx and a caller-side workspace tensor."""

    def __init__(self, d, n_qh, n_kvh, d_h, in_dtype=torch.bfloat16, out_dtype=torch.bfloat16):
        self._L = lib()
        self.handle = C.c_void_p()
        self.in_dtype, self.out_dtype = in_dtype, out_dtype
        self.d, self.n_qh, self.n_kvh, self.d_h = d, n_qh, n_kvh, d_h
        _check(None, self._L.pact_create(C.byref(self.handle), d, n_qh, n_kvh, d_h, _dt(in_dtype), _dt(out_dtype)))
        self.ws = None

    def close(self):
        if self.handle:
            self._L.pact_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def workspace_bytes(self, max_batch, max_N) -> int:
        return int(self._L.pact_workspace_bytes(self.handle, max_batch, max_N))

    def ensure_workspace(self, max_batch, max_N):
        need = self.workspace_bytes(max_batch, max_N)
        if self.ws is None or self.ws.numel() < need:
            self.ws = torch.empty(need, dtype=torch.uint8, device="cuda")
        return self.ws

    def _ws(self):
        return C.c_void_p(self.ws.data_ptr()), C.c_size_t(self.ws.numel())

    # ---- stage calls ------------------------------------------------------------------
    def pact_importance(self, im: DeviceImage, params: Params, score: torch.Tensor):
        self.ensure_workspace(1, im.N)
        d = im.desc()
        w, n = self._ws()
        _check(self.handle, self._L.pact_importance(self.handle, C.byref(d), C.byref(params), _ptr(score), w, n, _stream()))

    def pact_prune(self, score, params: Params, keep, kept_idx, pruned_idx, counts):
        N = score.numel()
        self.ensure_workspace(1, N)
        w, n = self._ws()
        _check(self.handle, self._L.pact_prune(self.handle, _ptr(score), N, C.byref(params), _ptr(keep),
                                               _ptr(kept_idx), _ptr(pruned_idx), _ptr(counts), w, n, _stream()))

    def pact_dbdpc(self, K, idx, q_dev, params: Params, rho, center_idx, C_dev, label, counters=None):
        N = K.shape[0]
        self.ensure_workspace(1, N)
        w, n = self._ws()
        _check(self.handle, self._L.pact_dbdpc(self.handle, _ptr(K), K.stride(0), N, _ptr(idx), _ptr(q_dev),
                                               C.byref(params), _ptr(rho), _ptr(center_idx), _ptr(C_dev),
                                               _ptr(label), _ptr(counters), w, n, _stream()))

    def pact_reincorporate(self, K, pruned_idx, m_dev, center_idx, C_dev, params: Params, label, r_dev,
                           counters=None):
        N = K.shape[0]
        self.ensure_workspace(1, N)
        w, n = self._ws()
        _check(self.handle, self._L.pact_reincorporate(self.handle, _ptr(K), K.stride(0), N, _ptr(pruned_idx),
                                                       _ptr(m_dev), _ptr(center_idx), _ptr(C_dev),
                                                       C.byref(params), _ptr(label), _ptr(r_dev),
                                                       _ptr(counters), w, n, _stream()))

    def pact_key_spread(self, K_layers, threshold: float, max_dist, layer_out=None):
        """K_layers: list of [N, d_k] key matrices (same N and row stride), one per layer."""
        N, ld = K_layers[0].shape[0], K_layers[0].stride(0)
        assert all(K.shape[0] == N and K.stride(0) == ld for K in K_layers)
        self.ensure_workspace(min(len(K_layers), 16), N)
        arr = (C.c_void_p * len(K_layers))(*[K.data_ptr() for K in K_layers])
        w, n = self._ws()
        _check(self.handle, self._L.pact_key_spread(self.handle, arr, len(K_layers), ld, N, float(threshold),
                                                    _ptr(max_dist), _ptr(layer_out), w, n, _stream()))

    def pact_merge(self, im: DeviceImage, label, center_idx, C_dev, params: Params):
        self.ensure_workspace(1, im.N)
        d = im.desc()
        w, n = self._ws()
        _check(self.handle, self._L.pact_merge(self.handle, C.byref(d), _ptr(label), _ptr(center_idx),
                                               _ptr(C_dev), C.byref(params), w, n, _stream()))

    # ---- the whole step -----------------------------------------------------------------
    def pact_reduce(self, images, params):
        """images: list of DeviceImage; params: one Params or a list with one per image."""
        B = len(images)
        self.ensure_workspace(B, max(im.N for im in images))
        arr = (ImageDesc * B)(*[im.desc() for im in images])
        if isinstance(params, Params):
            parr, stride = (Params * 1)(params), 0
        else:
            parr, stride = (Params * B)(*params), 1
        w, n = self._ws()
        _check(self.handle, self._L.pact_reduce(self.handle, arr, B, parr, stride, w, n, _stream()))

    def pact_graph_create(self, images, params):
        """Records pact_reduce(images, params) as a replayable graph (see Graph)."""
        B = len(images)
        self.ensure_workspace(B, max(im.N for im in images))
        arr = (ImageDesc * B)(*[im.desc() for im in images])
        if isinstance(params, Params):
            parr, stride = (Params * 1)(params), 0
        else:
            parr, stride = (Params * B)(*params), 1
        w, n = self._ws()
        h = C.c_void_p()
        _check(self.handle, self._L.pact_graph_create(self.handle, arr, B, parr, stride, w, n, C.byref(h)))
        return Graph(self, h, images, self.ws)

    def set_wait_limits(self, barrier_polls: int = 0, center_sweeps: int = 0):
        """Bounds of the device-side waits (0 = default); see pact_set_wait_limits in pact.h."""
        _check(self.handle, self._L.pact_set_wait_limits(self.handle, int(barrier_polls), int(center_sweeps)))

    def launch_count(self) -> int:
        return int(self._L.pact_launch_count(self.handle))

    def profile_enable(self, on: bool):
        _check(self.handle, self._L.pact_profile_enable(self.handle, 1 if on else 0))

    def profile_read(self) -> dict:
        """Per-kernel milliseconds of the last profiled pact_reduce (waits for it to finish)."""
        buf = (C.c_float * 16)()
        n = self._L.pact_profile_read(self.handle, buf, 16)
        return {self._L.pact_profile_stage_name(i).decode(): float(buf[i]) for i in range(n)}

    def host_staging_bytes(self, n_total, N) -> int:
        return int(self._L.pact_host_staging_bytes(self.handle, n_total, N))

    def pact_reduce_host(self, host: dict, params: Params, staging: torch.Tensor):
        """host: dict of pinned CPU tensors H, K_euti, Q_euti, K_clu, P, H_out, P_out, size_out,
        label, counters (and optionally logw_out) plus vis_start, N.  Copies in, reduces, copies the valid rows out."""
        self.ensure_workspace(1, host["N"])
        H = host["H"]
        d = ImageDesc(_ptr(H), H.stride(0), _ptr(host["K_euti"]), host["K_euti"].stride(0),
                      _ptr(host["Q_euti"]), host["Q_euti"].stride(0), _ptr(host["K_clu"]),
                      host["K_clu"].stride(0), _ptr(host["P"]), H.shape[0], host["vis_start"], host["N"], 0,
                      _ptr(host["H_out"]), host["H_out"].stride(0), _ptr(host["P_out"]),
                      _ptr(host["size_out"]), _ptr(host.get("label")), None, None, _ptr(host["counters"]),
                      _ptr(host.get("logw_out")))
        w, n = self._ws()
        _check(self.handle, self._L.pact_reduce_host(self.handle, C.byref(d), C.byref(params),
                                                     _ptr(staging), C.c_size_t(staging.numel()), w, n, _stream()))

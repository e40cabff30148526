"""ctypes binding of libla_b200.so: argument marshalling only.

The methods carry the names of the C entry points declared in include/la.h and take torch
tensors where the C side takes device pointers.  Every step of the layer runs inside the
library's CUDA kernels; torch supplies device memory and streams.  There is no fallback: if the
shared library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libla_b200.so")
_lib = None

LA_OK, LA_ERR_INVALID_ARG, LA_ERR_UNSUPPORTED, LA_ERR_CUDA, LA_ERR_BAD_TREE, LA_ERR_TIMEOUT, LA_ERR_TOO_LARGE = range(7)
LA_PHI = {"elu1": 0, "relu": 1}
LA_DTYPE = {"f32": 0, "bf16": 1}
TORCH_DTYPE = {"f32": torch.float32, "bf16": torch.bfloat16}
LA_MAX_TAPS, LA_MAX_NODES, LA_NOALLOC_MAX_SEQ = 32, 64, 1024

EXPORTS = ["la_create", "la_destroy", "la_status_str", "la_prefill", "la_decode_step", "la_verify_tree",
           "la_commit", "la_last_device_status", "la_clear_device_status", "la_set_prefill_kernel",
           "la_launch_count", "la_verify_tree_noalloc", "la_set_workspace", "la_accept_greedy", "la_selftest_wait_timeout",
           "la_prefill_workspace_bytes", "la_prefill_grouped", "la_prefill_grouped_max_group",
           "la_segment_state", "la_state_prefix", "la_accept_threshold"]


class LaError(RuntimeError):
    def __init__(self, fn: str, code: int):
        self.code = code
        super().__init__(f"{fn} failed: {status_str(code)} ({code})")


class la_config(C.Structure):
    _fields_ = [("H", C.c_int32), ("d", C.c_int32), ("conv_taps", C.c_int32), ("chunk", C.c_int32),
                ("phi", C.c_int), ("eps", C.c_float), ("io_dtype", C.c_int), ("max_nodes", C.c_int32),
                ("max_depth", C.c_int32)]


class la_state(C.Structure):
    _fields_ = [("S", C.c_void_p), ("z", C.c_void_p), ("win", C.c_void_p), ("pos", C.c_void_p)]


def lib() -> C.CDLL:
    """Loads the shared library once; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(f"{_LIB_PATH} is missing: build it with `python -m paper_2406_07368_b200.build` "
                               "(there is no CPU or eager fallback)")
        L = C.CDLL(_LIB_PATH)
        vp, i32 = C.c_void_p, C.c_int32
        L.la_create.argtypes = [C.POINTER(la_config), C.POINTER(vp)]
        L.la_destroy.argtypes = [vp]
        L.la_status_str.argtypes = [C.c_int]
        L.la_status_str.restype = C.c_char_p
        L.la_prefill.argtypes = [vp, i32, i32, vp, vp, vp, vp, i32, C.POINTER(la_state), vp, vp]
        L.la_prefill_grouped.argtypes = [vp, i32, i32, vp, vp, vp, vp, i32, C.c_float, C.c_float, i32, C.POINTER(la_state),
                                         vp, vp]
        L.la_prefill_grouped_max_group.argtypes = [vp]
        L.la_prefill_grouped_max_group.restype = i32
        L.la_segment_state.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp]
        L.la_state_prefix.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp]
        L.la_decode_step.argtypes = [vp, i32, vp, vp, vp, vp, C.POINTER(la_state), vp, vp]
        L.la_verify_tree.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp, C.POINTER(la_state), vp, vp]
        L.la_commit.argtypes = [vp, i32, i32, vp, vp, vp, vp, C.POINTER(la_state), vp, vp, vp]
        L.la_accept_greedy.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp]
        L.la_accept_threshold.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp, vp]
        L.la_selftest_wait_timeout.argtypes = [vp, C.c_uint32, vp, vp]
        L.la_verify_tree_noalloc.argtypes = [C.POINTER(la_config), i32, i32, vp, vp, vp, vp, vp, C.POINTER(la_state),
                                             vp, vp, vp]
        L.la_last_device_status.argtypes = [vp, vp]
        L.la_clear_device_status.argtypes = [vp, vp]
        L.la_set_prefill_kernel.argtypes = [vp, i32]
        L.la_launch_count.argtypes = [vp]
        L.la_set_workspace.argtypes = [vp, vp, C.c_uint64]
        L.la_prefill_workspace_bytes.argtypes = [vp, i32, i32]
        L.la_prefill_workspace_bytes.restype = C.c_uint64
        L.la_launch_count.restype = C.c_int64
        for name in EXPORTS:
            if name not in ("la_status_str", "la_launch_count", "la_prefill_workspace_bytes", "la_prefill_grouped_max_group"):
                getattr(L, name).restype = C.c_int
        _lib = L
    return _lib


def status_str(code: int) -> str:
    return lib().la_status_str(int(code)).decode()


def _check(fn: str, code: int) -> None:
    if code != LA_OK:
        raise LaError(fn, code)


def _ptr(t, dtype=None, shape=None, name="tensor"):
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError(f"{name} must be a contiguous CUDA tensor")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"{name} must have dtype {dtype}, got {t.dtype}")
    if shape is not None and tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name} must have shape {tuple(shape)}, got {tuple(t.shape)}")
    return t.data_ptr()


def _stream(stream) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


@dataclass
class State:
    """Caller-owned running state of B sequences (see la_state in include/la.h)."""
    S: torch.Tensor      # [B, H, d, d] fp32
    z: torch.Tensor      # [B, H, d] fp32
    win: torch.Tensor    # [B, H, W-1, d] io type
    pos: torch.Tensor    # [B] int64

    def c(self) -> la_state:
        return la_state(self.S.data_ptr(), self.z.data_ptr(), self.win.data_ptr() if self.win.numel() else None,
                        self.pos.data_ptr())

    def clone(self) -> "State":
        return State(self.S.clone(), self.z.clone(), self.win.clone(), self.pos.clone())


class Context:
    """Owns an la_ctx*.  Methods are named after the C entry points."""

    def __init__(self, H: int, d: int, conv_taps: int, phi: str = "elu1", eps: float = 0.0, io: str = "bf16",
                 chunk: int = 0, max_nodes: int = 64, max_depth: int = 8, device: int | None = None):
        self.H, self.d, self.W, self.io = H, d, conv_taps, io
        self.max_nodes, self.max_depth = max_nodes, max_depth
        self.dtype = TORCH_DTYPE[io]
        self.device = torch.device("cuda", torch.cuda.current_device() if device is None else device)
        self._h = C.c_void_p()
        cfg = la_config(H, d, conv_taps, chunk, LA_PHI[phi], eps, LA_DTYPE[io], max_nodes, max_depth)
        with torch.cuda.device(self.device):
            torch.cuda.current_stream()          # make sure the device context exists
            _check("la_create", lib().la_create(C.byref(cfg), C.byref(self._h)))

    def close(self) -> None:
        if self._h:
            lib().la_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- state helpers (device memory only) ------------------------------------------------
    def new_state(self, B: int) -> State:
        dev = self.device
        return State(torch.zeros(B, self.H, self.d, self.d, dtype=torch.float32, device=dev),
                     torch.zeros(B, self.H, self.d, dtype=torch.float32, device=dev),
                     torch.zeros(B, self.H, self.W - 1, self.d, dtype=self.dtype, device=dev),
                     torch.zeros(B, dtype=torch.int64, device=dev))

    def _check_state(self, st: State, B: int) -> None:
        _ptr(st.S, torch.float32, (B, self.H, self.d, self.d), "state.S")
        _ptr(st.z, torch.float32, (B, self.H, self.d), "state.z")
        _ptr(st.win, self.dtype, (B, self.H, self.W - 1, self.d), "state.win")
        _ptr(st.pos, torch.int64, (B,), "state.pos")

    # -- entry points ----------------------------------------------------------------------
    def la_prefill(self, q, k, v, conv_w, state: State, init_state: bool = False, out=None, stream=None):
        B, H, T, d = q.shape
        shp = (B, self.H, T, self.d)
        out = torch.empty(shp, dtype=self.dtype, device=q.device) if out is None else out
        self._check_state(state, B)
        cs = state.c()
        _check("la_prefill", lib().la_prefill(
            self._h, B, T, _ptr(q, self.dtype, shp, "q"), _ptr(k, self.dtype, shp, "k"), _ptr(v, self.dtype, shp, "v"),
            _ptr(conv_w, torch.float32, (self.H, self.d, self.W), "conv_w"), int(bool(init_state)), C.byref(cs),
            _ptr(out, self.dtype, shp, "o"), _stream(stream)))
        return out

    def la_prefill_grouped(self, q, k, v, conv_w, state: State, group: int, alpha: float, softmax_scale: float,
                           init_state: bool = False, out=None, stream=None):
        B, H, T, d = q.shape
        shp = (B, self.H, T, self.d)
        out = torch.empty(shp, dtype=self.dtype, device=q.device) if out is None else out
        self._check_state(state, B)
        cs = state.c()
        _check("la_prefill_grouped", lib().la_prefill_grouped(
            self._h, B, T, _ptr(q, self.dtype, shp, "q"), _ptr(k, self.dtype, shp, "k"), _ptr(v, self.dtype, shp, "v"),
            _ptr(conv_w, torch.float32, (self.H, self.d, self.W), "conv_w"), int(group), float(alpha),
            float(softmax_scale), int(bool(init_state)), C.byref(cs), _ptr(out, self.dtype, shp, "o"), _stream(stream)))
        return out

    def la_prefill_grouped_max_group(self) -> int:
        return int(lib().la_prefill_grouped_max_group(self._h))

    def la_segment_state(self, k, v, dS=None, dz=None, stream=None):
        """Sums of one stretch of the sequence: (dS [B,H,d,d], dz [B,H,d]) fp32."""
        B, H, T, d = k.shape
        shp = (B, self.H, T, self.d)
        dS = torch.empty(B, self.H, self.d, self.d, dtype=torch.float32, device=k.device) if dS is None else dS
        dz = torch.empty(B, self.H, self.d, dtype=torch.float32, device=k.device) if dz is None else dz
        _check("la_segment_state", lib().la_segment_state(
            self._h, B, T, _ptr(k, self.dtype, shp, "k"), _ptr(v, self.dtype, shp, "v"),
            _ptr(dS, torch.float32, (B, self.H, self.d, self.d), "dS"), _ptr(dz, torch.float32, (B, self.H, self.d), "dz"),
            _stream(stream)))
        return dS, dz

    def la_state_prefix(self, dS_parts, dz_parts, count: int, S_base=None, z_base=None, stream=None):
        """S_base + the first `count` parts of dS_parts [nparts,B,H,d,d] (likewise z): returns (S, z)."""
        nparts, B = dS_parts.shape[0], dS_parts.shape[1]
        S = torch.empty(dS_parts.shape[1:], dtype=torch.float32, device=dS_parts.device)
        z = torch.empty(dz_parts.shape[1:], dtype=torch.float32, device=dz_parts.device)
        _check("la_state_prefix", lib().la_state_prefix(
            self._h, B, nparts, int(count), _ptr(dS_parts, torch.float32, (nparts, B, self.H, self.d, self.d), "dS_parts"),
            _ptr(dz_parts, torch.float32, (nparts, B, self.H, self.d), "dz_parts"),
            _ptr(S_base, torch.float32, (B, self.H, self.d, self.d), "S_base"),
            _ptr(z_base, torch.float32, (B, self.H, self.d), "z_base"), S.data_ptr(), z.data_ptr(), _stream(stream)))
        return S, z

    def la_decode_step(self, q, k, v, conv_w, state: State, out=None, stream=None):
        B = q.shape[0]
        shp = (B, self.H, self.d)
        out = torch.empty(shp, dtype=self.dtype, device=q.device) if out is None else out
        self._check_state(state, B)
        cs = state.c()
        _check("la_decode_step", lib().la_decode_step(
            self._h, B, _ptr(q, self.dtype, shp, "q"), _ptr(k, self.dtype, shp, "k"), _ptr(v, self.dtype, shp, "v"),
            _ptr(conv_w, torch.float32, (self.H, self.d, self.W), "conv_w"), C.byref(cs),
            _ptr(out, self.dtype, shp, "o"), _stream(stream)))
        return out

    def la_verify_tree(self, q, k, v, parent, conv_w, state: State, out=None, stream=None):
        B, H, N, d = q.shape
        shp = (B, self.H, N, self.d)
        out = torch.empty(shp, dtype=self.dtype, device=q.device) if out is None else out
        self._check_state(state, B)
        cs = state.c()
        _check("la_verify_tree", lib().la_verify_tree(
            self._h, B, N, _ptr(q, self.dtype, shp, "q"), _ptr(k, self.dtype, shp, "k"), _ptr(v, self.dtype, shp, "v"),
            _ptr(parent, torch.int32, (B, N), "parent"),
            _ptr(conv_w, torch.float32, (self.H, self.d, self.W), "conv_w"), C.byref(cs),
            _ptr(out, self.dtype, shp, "o"), _stream(stream)))
        return out

    def la_commit(self, k, v, parent, accept_node, state: State, path_out=None, commit_len=None, stream=None):
        B, H, N, d = k.shape
        shp = (B, self.H, N, self.d)
        if path_out is None:
            path_out = torch.full((B, self.max_depth), -1, dtype=torch.int32, device=k.device)
        if commit_len is None:
            commit_len = torch.zeros(B, dtype=torch.int32, device=k.device)
        self._check_state(state, B)
        cs = state.c()
        _check("la_commit", lib().la_commit(
            self._h, B, N, _ptr(k, self.dtype, shp, "k"), _ptr(v, self.dtype, shp, "v"),
            _ptr(parent, torch.int32, (B, N), "parent"), _ptr(accept_node, torch.int32, (B,), "accept_node"),
            C.byref(cs), _ptr(path_out, torch.int32, (B, self.max_depth), "path_out"),
            _ptr(commit_len, torch.int32, (B,), "commit_len"), _stream(stream)))
        return path_out, commit_len

    def la_accept_greedy(self, parent, draft_token, pred_root, pred, accept_node=None, accept_len=None,
                         next_token=None, stream=None):
        B, N = parent.shape
        dev = parent.device
        accept_node = torch.empty(B, dtype=torch.int32, device=dev) if accept_node is None else accept_node
        accept_len = torch.empty(B, dtype=torch.int32, device=dev) if accept_len is None else accept_len
        next_token = torch.empty(B, dtype=torch.int32, device=dev) if next_token is None else next_token
        _check("la_accept_greedy", lib().la_accept_greedy(
            self._h, B, N, _ptr(parent, torch.int32, (B, N), "parent"),
            _ptr(draft_token, torch.int32, (B, N), "draft_token"), _ptr(pred_root, torch.int32, (B,), "pred_root"),
            _ptr(pred, torch.int32, (B, N), "pred"), _ptr(accept_node, torch.int32, (B,), "accept_node"),
            _ptr(accept_len, torch.int32, (B,), "accept_len"), _ptr(next_token, torch.int32, (B,), "next_token"),
            _stream(stream)))
        return accept_node, accept_len, next_token

    def la_accept_threshold(self, parent, score, thresh, accept_node=None, accept_len=None, stream=None):
        B, N = parent.shape
        dev = parent.device
        accept_node = torch.empty(B, dtype=torch.int32, device=dev) if accept_node is None else accept_node
        accept_len = torch.empty(B, dtype=torch.int32, device=dev) if accept_len is None else accept_len
        _check("la_accept_threshold", lib().la_accept_threshold(
            self._h, B, N, _ptr(parent, torch.int32, (B, N), "parent"), _ptr(score, torch.float32, (B, N), "score"),
            _ptr(thresh, torch.float32, (B, N), "thresh"), _ptr(accept_node, torch.int32, (B,), "accept_node"),
            _ptr(accept_len, torch.int32, (B,), "accept_len"), _stream(stream)))
        return accept_node, accept_len

    def la_selftest_wait_timeout(self, limit_us: int, stream=None) -> int:
        """Runs the bounded-wait self-test; returns the nanoseconds the wait took (see include/la.h)."""
        waited = torch.zeros(1, dtype=torch.int64, device="cuda")
        _check("la_selftest_wait_timeout", lib().la_selftest_wait_timeout(self._h, int(limit_us), waited.data_ptr(),
                                                                          _stream(stream)))
        return int(waited.item())

    def la_last_device_status(self, stream=None) -> int:
        return int(lib().la_last_device_status(self._h, _stream(stream)))

    def la_clear_device_status(self, stream=None) -> None:
        _check("la_clear_device_status", lib().la_clear_device_status(self._h, _stream(stream)))

    def la_set_prefill_kernel(self, which: int) -> None:
        _check("la_set_prefill_kernel", lib().la_set_prefill_kernel(self._h, which))

    def la_launch_count(self) -> int:
        return int(lib().la_launch_count(self._h))

    def la_prefill_workspace_bytes(self, B: int, T: int) -> int:
        return int(lib().la_prefill_workspace_bytes(self._h, B, T))

    def la_set_workspace(self, workspace: torch.Tensor | None) -> None:
        """Lends a device buffer (any dtype, contiguous) to the context; it is kept alive by this object."""
        self._ws = workspace
        if workspace is None:
            _check("la_set_workspace", lib().la_set_workspace(self._h, None, 0))
        else:
            _check("la_set_workspace", lib().la_set_workspace(self._h, _ptr(workspace, name="workspace"),
                                                              workspace.numel() * workspace.element_size()))


def la_verify_tree_noalloc(H: int, d: int, conv_taps: int, phi: str, eps: float, io: str, q, k, v, parent, conv_w,
                           state: State, out, seq_status=None, stream=None) -> None:
    """Tree verification without a context, for callers that are not allowed to allocate.

    Every buffer, including `out` ([B, H, N, d]) and the optional per-sequence status
    `seq_status` ([B] int32), is supplied by the caller; neither this wrapper nor the C entry
    point behind it allocates device memory.  See la_verify_tree_noalloc in include/la.h for
    the batch limit and the rule about overlapping calls.
    """
    B, _, N, _ = q.shape
    dt = TORCH_DTYPE[io]
    shp = (B, H, N, d)
    cfg = la_config(H, d, conv_taps, 0, LA_PHI[phi], eps, LA_DTYPE[io], LA_MAX_NODES, LA_MAX_NODES)
    cs = state.c()
    _check("la_verify_tree_noalloc", lib().la_verify_tree_noalloc(
        C.byref(cfg), B, N, _ptr(q, dt, shp, "q"), _ptr(k, dt, shp, "k"), _ptr(v, dt, shp, "v"),
        _ptr(parent, torch.int32, (B, N), "parent"), _ptr(conv_w, torch.float32, (H, d, conv_taps), "conv_w"),
        C.byref(cs), _ptr(out, dt, shp, "o"), _ptr(seq_status, torch.int32, (B,), "seq_status"), _stream(stream)))

"""ctypes binding of libsr_rollout.so (see include/sr_rollout.h for the contract).

Argument marshalling only.  PyTorch provides device memory and streams; there is
no fallback: if the library cannot be loaded, or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libsr_rollout.so")
_lib = None

STATUS = {0: "SR_OK", 1: "SR_ERR_INVALID_ARG", 2: "SR_ERR_NOT_A_NETWORK", 3: "SR_ERR_INVALID_ROLLOUT",
          4: "SR_ERR_SHAPE_MISMATCH", 5: "SR_ERR_UNSUPPORTED", 6: "SR_ERR_CUDA", 7: "SR_ERR_TIMEOUT", 8: "SR_ERR_STATE",
          9: "SR_ERR_TOO_LARGE"}


class SrError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        self.status = STATUS.get(code, "?")
        super().__init__("%s: %s (%s)" % (what, self.status, _status_str(code)))


class _NodeDesc(ctypes.Structure):
    _fields_ = [("h", ctypes.c_int32), ("w", ctypes.c_int32), ("c", ctypes.c_int32), ("act", ctypes.c_int32)]


class _EdgeDesc(ctypes.Structure):
    _fields_ = [("src", ctypes.c_int32), ("tgt", ctypes.c_int32), ("kind", ctypes.c_int32),
                ("k", ctypes.c_int32), ("stride", ctypes.c_int32), ("pool", ctypes.c_int32)]


class _Info(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("n_nodes", "n_edges", "n_inputs", "inference_factor", "n_groups", "streaming_parallel",
                 "output_node", "first_response_frame", "first_response_step", "response_interval",
                 "n_tensor_core_nodes", "n_direct_nodes", "resident_cluster", "resident_smem_bytes", "resident_heads_on_chip")]


def load_library(path: Optional[str] = None):
    """Load the C-ABI library; build it first if the file is missing and nvcc is present."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or _LIB_PATH
    if not os.path.exists(p):
        from . import build as _build
        _build.build()
    lib = ctypes.CDLL(p)
    vp, ip = ctypes.c_void_p, ctypes.c_int
    lib.sr_graph_create.argtypes = [ctypes.POINTER(_NodeDesc), ip, ctypes.POINTER(_EdgeDesc), ip,
                                    ctypes.POINTER(ctypes.c_uint8), ip, ip, ctypes.POINTER(vp)]
    lib.sr_graph_destroy.argtypes = [vp]
    lib.sr_graph_destroy.restype = None
    lib.sr_graph_info.argtypes = [vp, ctypes.POINTER(_Info)]
    lib.sr_graph_levels.argtypes = [vp, ctypes.POINTER(ctypes.c_int32)]
    lib.sr_graph_workspace_bytes.argtypes = [vp, ctypes.POINTER(ctypes.c_size_t)]
    lib.sr_graph_bind_workspace.argtypes = [vp, vp, ctypes.c_size_t]
    lib.sr_graph_bind_static_workspace.argtypes = [vp]
    lib.sr_graph_bind_static_workspace.restype = ctypes.c_int
    lib.sr_graph_set_edge_weights.argtypes = [vp, ip, vp, ip]
    lib.sr_graph_set_node_bias.argtypes = [vp, ip, vp]
    lib.sr_graph_set_option.argtypes = [vp, ip, ip]
    lib.sr_graph_reset.argtypes = [vp, ctypes.POINTER(vp), vp]
    lib.sr_rollout_step.argtypes = [vp, ctypes.POINTER(vp), vp, vp]
    lib.sr_rollout_run.argtypes = [vp, ctypes.POINTER(vp), ip, vp, vp]
    lib.sr_graph_get_state.argtypes = [vp, ip, vp, vp]
    lib.sr_graph_set_state.argtypes = [vp, ip, vp, vp]
    lib.sr_graph_frame.argtypes = [vp, ctypes.POINTER(ctypes.c_int64)]
    lib.sr_graph_launch_count.argtypes = [vp, ctypes.POINTER(ctypes.c_int64)]
    lib.sr_graph_sync_status.argtypes = [vp, vp]
    lib.sr_graph_kernel_time.argtypes = [vp, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_int64)]
    lib.sr_graph_kernel_time.restype = ctypes.c_int
    lib.sr_graph_window_tableau.argtypes = [vp, ip, ctypes.POINTER(ctypes.c_int32)]
    lib.sr_graph_window_workspace_bytes.argtypes = [vp, ip, ctypes.POINTER(ctypes.c_size_t)]
    lib.sr_graph_bind_window.argtypes = [vp, ip, vp, ctypes.c_size_t]
    lib.sr_rollout_window.argtypes = [vp, ctypes.POINTER(vp), ip, vp, vp]
    for name in ("sr_graph_window_tableau", "sr_graph_window_workspace_bytes", "sr_graph_bind_window", "sr_rollout_window"):
        getattr(lib, name).restype = ctypes.c_int
    lib.sr_status_str.argtypes = [ip]
    lib.sr_status_str.restype = ctypes.c_char_p
    for name in ("sr_graph_create", "sr_graph_info", "sr_graph_levels", "sr_graph_workspace_bytes",
                 "sr_graph_bind_workspace", "sr_graph_set_edge_weights", "sr_graph_set_node_bias",
                 "sr_graph_set_option", "sr_graph_reset", "sr_rollout_step", "sr_rollout_run", "sr_graph_get_state",
                 "sr_graph_set_state", "sr_graph_frame", "sr_graph_launch_count", "sr_graph_sync_status"):
        getattr(lib, name).restype = ctypes.c_int
    if path is None:
        _lib = lib
    return lib


def _status_str(code: int) -> str:
    try:
        return load_library().sr_status_str(code).decode()
    except Exception:
        return "?"


def _check(code: int, what: str):
    if code != 0:
        raise SrError(code, what)


class Graph:
    """A compiled network + rollout pattern (sr_graph).  batch=0 gives a theory-only graph."""

    def __init__(self, nodes: Sequence, edges: Sequence, R: Sequence[int], batch: int = 0, dtype: str = "bf16",
                 engine: str = "auto", graph_frames: int = 0, device: str = "cuda:0", static_workspace: bool = False, weight_ring_units: int = 0, tile_width: int = 0,
                 resident: bool = True, resident_cluster: int = 0, resident_warps: int = 0, resident_split: int = 0,
                 wait_limit_ms: Optional[int] = None, tc_pair: int = 0, stem_ring: int = 1, tc_lists: int = 0, tc_fuse: int = 1):
        self._lib = load_library()
        self._h = ctypes.c_void_p()
        self.nodes, self.edges, self.R = list(nodes), list(edges), [int(r) for r in R]
        self.batch, self.dtype = batch, dtype
        n, m = len(self.nodes), len(self.edges)
        cn = (_NodeDesc * max(n, 1))(*[_NodeDesc(v.h, v.w, v.c, v.act) for v in self.nodes])
        ce = (_EdgeDesc * max(m, 1))(*[_EdgeDesc(e.src, e.tgt, e.kind, e.k, e.stride, e.pool) for e in self.edges])
        cr = (ctypes.c_uint8 * max(m, 1))(*self.R)
        _check(self._lib.sr_graph_create(cn, n, ce, m, cr, batch, {"fp32": 0, "bf16": 1}[dtype],
                                         ctypes.byref(self._h)), "sr_graph_create")
        self._ws = None
        self._keep = []
        self.device = device
        if batch > 0:
            import torch
            if not torch.cuda.is_available():
                raise RuntimeError("a CUDA device is required for a graph with batch > 0")
            self._torch = torch
            self.tdtype = torch.bfloat16 if dtype == "bf16" else torch.float32
            _check(self._lib.sr_graph_set_option(self._h, 0, {"auto": 0, "direct": 1}[engine]), "sr_graph_set_option")
            _check(self._lib.sr_graph_set_option(self._h, 1, int(graph_frames)), "sr_graph_set_option")
            _check(self._lib.sr_graph_set_option(self._h, 2, int(weight_ring_units)), "sr_graph_set_option")
            _check(self._lib.sr_graph_set_option(self._h, 3, int(tile_width)), "sr_graph_set_option")
            _check(self._lib.sr_graph_set_option(self._h, 6, 1 if resident else 0), "sr_graph_set_option")
            _check(self._lib.sr_graph_set_option(self._h, 7, int(resident_cluster)), "sr_graph_set_option")
            _check(self._lib.sr_graph_set_option(self._h, 8, int(resident_warps)), "sr_graph_set_option")
            _check(self._lib.sr_graph_set_option(self._h, 9, int(resident_split)), "sr_graph_set_option")
            if wait_limit_ms is not None:
                _check(self._lib.sr_graph_set_option(self._h, 10, int(wait_limit_ms)), "sr_graph_set_option")
            _check(self._lib.sr_graph_set_option(self._h, 11, int(tc_pair)), "sr_graph_set_option")
            _check(self._lib.sr_graph_set_option(self._h, 12, int(stem_ring)), "sr_graph_set_option")
            _check(self._lib.sr_graph_set_option(self._h, 13, int(tc_lists)), "sr_graph_set_option")
            _check(self._lib.sr_graph_set_option(self._h, 14, int(tc_fuse)), "sr_graph_set_option")
            nbytes = ctypes.c_size_t()
            _check(self._lib.sr_graph_workspace_bytes(self._h, ctypes.byref(nbytes)), "sr_graph_workspace_bytes")
            self.workspace_bytes = nbytes.value
            if static_workspace:
                # the library's built-in array serves as workspace: no device allocation for the graph
                _check(self._lib.sr_graph_bind_static_workspace(self._h), "sr_graph_bind_static_workspace")
            else:
                self._ws = torch.empty(nbytes.value + 256, dtype=torch.uint8, device=device)
                base = (self._ws.data_ptr() + 255) // 256 * 256
                _check(self._lib.sr_graph_bind_workspace(self._h, base, nbytes.value), "sr_graph_bind_workspace")
        self.info = self._info()
        self.input_nodes = [v for v in range(n) if not any(e.tgt == v for e in self.edges)]
        self.output_node = self.info["output_node"]

    def __del__(self):
        try:
            if self._h:
                self._lib.sr_graph_destroy(self._h)
                self._h = None
        except Exception:
            pass

    def _info(self) -> dict:
        i = _Info()
        _check(self._lib.sr_graph_info(self._h, ctypes.byref(i)), "sr_graph_info")
        return {n: getattr(i, n) for (n, _) in _Info._fields_}

    def levels(self) -> List[int]:
        lv = (ctypes.c_int32 * len(self.nodes))()
        _check(self._lib.sr_graph_levels(self._h, lv), "sr_graph_levels")
        return list(lv)

    def _stream(self):
        return self._torch.cuda.current_stream().cuda_stream

    def set_weights(self, weights: Sequence[np.ndarray], biases: Optional[Sequence[np.ndarray]] = None):
        for ei, w in enumerate(weights):
            w = np.ascontiguousarray(w, dtype=np.float32)
            _check(self._lib.sr_graph_set_edge_weights(self._h, ei, w.ctypes.data, 0), "sr_graph_set_edge_weights")
        if biases is not None:
            for vi, b in enumerate(biases):
                b = np.ascontiguousarray(b, dtype=np.float32)
                _check(self._lib.sr_graph_set_node_bias(self._h, vi, b.ctypes.data), "sr_graph_set_node_bias")

    def _ptrs(self, tensors, frames: Optional[int] = None):
        assert len(tensors) == len(self.input_nodes)
        arr = (ctypes.c_void_p * len(tensors))()
        for i, (t, v) in enumerate(zip(tensors, self.input_nodes)):
            nd = self.nodes[v]
            shape = (self.batch, nd.h, nd.w, nd.c) if frames is None else (frames, self.batch, nd.h, nd.w, nd.c)
            assert t.is_cuda and t.is_contiguous() and t.dtype == self.tdtype and tuple(t.shape) == shape, (t.shape, shape)
            arr[i] = t.data_ptr()
        return arr

    def reset(self, in0):
        _check(self._lib.sr_graph_reset(self._h, self._ptrs(in0), self._stream()), "sr_graph_reset")

    def out_shape(self):
        """Shape of one frame of output: the output node's state, [B][C] for a dense node, else [B][H][W][C]."""
        nd = self.nodes[self.output_node]
        return (self.batch, nd.c) if nd.h == 1 and nd.w == 1 else (self.batch, nd.h, nd.w, nd.c)

    def step(self, in_next, out=None):
        if out is not None:
            assert out.is_cuda and out.is_contiguous() and out.dtype == self._torch.float32
            assert tuple(out.shape) == self.out_shape()
        _check(self._lib.sr_rollout_step(self._h, self._ptrs(in_next), out.data_ptr() if out is not None else None,
                                         self._stream()), "sr_rollout_step")

    def run(self, in_seq, out_seq=None):
        T = int(in_seq[0].shape[0])
        if out_seq is not None:
            assert out_seq.is_cuda and out_seq.is_contiguous() and out_seq.dtype == self._torch.float32
            assert tuple(out_seq.shape) == (T,) + self.out_shape()
        _check(self._lib.sr_rollout_run(self._h, self._ptrs(in_seq, T), T,
                                        out_seq.data_ptr() if out_seq is not None else None, self._stream()),
               "sr_rollout_run")

    def window_tableau(self, W: int) -> List[List[int]]:
        """T((i, v)) of the rollout window of size W, one row per frame i = 0..W (Eq. 4)."""
        n = len(self.nodes)
        buf = (ctypes.c_int32 * ((W + 1) * n))()
        _check(self._lib.sr_graph_window_tableau(self._h, W, buf), "sr_graph_window_tableau")
        return [list(buf[i * n:(i + 1) * n]) for i in range(W + 1)]

    def bind_window(self, W: int):
        """Allocates and binds the workspace of a window of W frames (after the parameters have been set)."""
        nbytes = ctypes.c_size_t()
        _check(self._lib.sr_graph_window_workspace_bytes(self._h, W, ctypes.byref(nbytes)), "sr_graph_window_workspace_bytes")
        self._window_ws = self._torch.empty(nbytes.value + 256, dtype=self._torch.uint8, device=self.device)
        base = (self._window_ws.data_ptr() + 255) // 256 * 256
        _check(self._lib.sr_graph_bind_window(self._h, W, base, nbytes.value), "sr_graph_bind_window")

    def rollout_window(self, in_seq, out_seq=None):
        """The W = in_seq[0].shape[0] frame updates t+1 .. t+W evaluated as one window."""
        W = int(in_seq[0].shape[0])
        if out_seq is not None:
            assert out_seq.is_cuda and out_seq.is_contiguous() and out_seq.dtype == self._torch.float32
            assert tuple(out_seq.shape) == (W,) + self.out_shape()
        _check(self._lib.sr_rollout_window(self._h, self._ptrs(in_seq, W), W,
                                           out_seq.data_ptr() if out_seq is not None else None, self._stream()),
               "sr_rollout_window")

    def get_state(self, node: int):
        nd = self.nodes[node]
        t = self._torch.empty((self.batch, nd.h, nd.w, nd.c), dtype=self.tdtype, device=self.device)
        _check(self._lib.sr_graph_get_state(self._h, node, t.data_ptr(), self._stream()), "sr_graph_get_state")
        return t

    def set_state(self, node: int, t):
        nd = self.nodes[node]
        assert t.is_cuda and t.is_contiguous() and t.dtype == self.tdtype
        assert tuple(t.shape) == (self.batch, nd.h, nd.w, nd.c)
        _check(self._lib.sr_graph_set_state(self._h, node, t.data_ptr(), self._stream()), "sr_graph_set_state")

    def frame(self) -> int:
        v = ctypes.c_int64()
        _check(self._lib.sr_graph_frame(self._h, ctypes.byref(v)), "sr_graph_frame")
        return v.value

    def launch_count(self) -> int:
        v = ctypes.c_int64()
        _check(self._lib.sr_graph_launch_count(self._h, ctypes.byref(v)), "sr_graph_launch_count")
        return v.value

    def set_option(self, key: int, value: int):
        _check(self._lib.sr_graph_set_option(self._h, key, value), "sr_graph_set_option")

    def kernel_time(self):
        """(milliseconds, launches) of the event-timed tensor-core group launches since the last call."""
        ms, n = ctypes.c_double(), ctypes.c_int64()
        _check(self._lib.sr_graph_kernel_time(self._h, ctypes.byref(ms), ctypes.byref(n)), "sr_graph_kernel_time")
        return ms.value, n.value

    def sync_status(self):
        _check(self._lib.sr_graph_sync_status(self._h, self._stream()), "sr_graph_sync_status")

    def rollout(self, frames):
        """frames: one tensor [T+1][B][H][W][C] per input node (frames 0..T).  Resets to frame 0,
        runs T updates, returns the outputs [T][B][C_out] (float32)."""
        T = int(frames[0].shape[0]) - 1
        out = self._torch.empty((T,) + self.out_shape(), dtype=self._torch.float32, device=self.device)
        self.reset([f[0] for f in frames])
        self.run([f[1:] for f in frames], out)
        return out

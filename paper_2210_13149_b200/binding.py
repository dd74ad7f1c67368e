"""ctypes binding of libbigcn (``include/bigcn.h``).

Argument marshalling only: every step of the forward path runs in the library's CUDA kernels.
torch is used for device memory (inputs, outputs, the workspace) and for the current stream.
There is no CPU fallback: if the shared library cannot be loaded or no CUDA device is present,
creating a :class:`BiGCN` raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import List, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libbigcn.so")

MAX_LAYERS = 16
OPT_ZETA_FORMAT = 1
OPT_LONG_ROW = 2
OPT_BYTE_AGGREGATION = 4   # rows of 129..256 bytes: 0 = default (3 where only bits and beta are wanted, else 1), 1 = fp32 FMA stream, 2 = integer products (mma.sync), 3 = integer products (tcgen05)
OPT_CONTRACTION = 3     # 0 = auto (default), 1 = XOR / bit-count pipe, 2 = tensor cores wherever the shape is covered
ZETA_AUTO, ZETA_F32, ZETA_I16, ZETA_I8, ZETA_F16, ZETA_I8H = 0, 1, 2, 3, 4, 5

_i32, _i64, _vp, _sz = ctypes.c_int32, ctypes.c_int64, ctypes.c_void_p, ctypes.c_size_t


class bigcn_graph(ctypes.Structure):
    _fields_ = [("n", _i64), ("nnz", _i64), ("rowptr", _vp), ("colidx", _vp), ("val", _vp), ("dinv", _vp)]


class bigcn_layer(ctypes.Structure):
    _fields_ = [("d_in", _i32), ("d_out", _i32), ("w_bitsT", _vp), ("alpha", _vp),
                ("in_shift", _vp), ("in_scale", _vp)]


class bigcn_stats(ctypes.Structure):
    _fields_ = [("n_layers", _i32), ("launches", _i32), ("ms_total", ctypes.c_float),
                ("ms_pack", ctypes.c_float), ("ms_gemm", ctypes.c_float * MAX_LAYERS),
                ("ms_spmm", ctypes.c_float * MAX_LAYERS)]


# name -> (restype, argtypes); every symbol include/bigcn.h declares
SIGNATURES = {
    "bigcn_create": (ctypes.c_int, [ctypes.POINTER(_vp), ctypes.c_int, _vp]),
    "bigcn_destroy": (ctypes.c_int, [_vp]),
    "bigcn_last_error": (ctypes.c_char_p, [_vp]),
    "bigcn_status_string": (ctypes.c_char_p, [ctypes.c_int]),
    "bigcn_set_option": (ctypes.c_int, [_vp, _i32, _i64]),
    "bigcn_launch_count": (_i64, [_vp]),
    "bigcn_sync_check": (ctypes.c_int, [_vp]),
    "bigcn_packed_stride_words": (_i64, [_i32]),
    "bigcn_workspace_bytes": (_sz, [_i64, _i64, ctypes.POINTER(_i32), _i32, _i32]),
    "bigcn_set_workspace": (ctypes.c_int, [_vp, _vp, _sz]),
    "bigcn_normalize_adjacency": (ctypes.c_int, [_vp, _i64, _i64, _vp, _vp, _vp, _vp, _vp, _vp,
                                                 ctypes.POINTER(_i64)]),
    "bigcn_edges_workspace_bytes": (_sz, [_i64, _i64]),
    "bigcn_adjacency_from_edges": (ctypes.c_int, [_vp, _i64, _i64, _vp, _vp, _vp, _vp, ctypes.POINTER(_i64)]),
    "bigcn_pack_features": (ctypes.c_int, [_vp, _vp, _i64, _i32, _i64, _vp, _vp, _vp, _i64, _vp]),
    "bigcn_pack_weights": (ctypes.c_int, [_vp, _vp, _i32, _i32, _i64, _vp, _i64, _vp]),
    "bigcn_layer_forward": (ctypes.c_int, [_vp, ctypes.POINTER(bigcn_graph), ctypes.POINTER(bigcn_layer),
                                           _vp, _vp, _vp, _i64, ctypes.POINTER(bigcn_layer), _vp, _vp, _vp, _vp]),
    "bigcn_forward": (ctypes.c_int, [_vp, ctypes.POINTER(bigcn_graph), ctypes.POINTER(bigcn_layer), _i32,
                                     _vp, _i64, _vp, _i64, ctypes.POINTER(bigcn_stats)]),
    "bigcn_forward_packed": (ctypes.c_int, [_vp, ctypes.POINTER(bigcn_graph), ctypes.POINTER(bigcn_layer), _i32,
                                            _vp, _vp, _vp, _i64, ctypes.POINTER(bigcn_stats)]),
    "bigcn_forward_host": (ctypes.c_int, [_vp, ctypes.POINTER(bigcn_graph), ctypes.POINTER(bigcn_layer), _i32,
                                          _vp, _i64, _vp, _i64]),
    "bigcn_pipeline_open": (ctypes.c_int, [_vp, ctypes.POINTER(bigcn_graph), ctypes.POINTER(bigcn_layer), _i32, _i32,
                                           ctypes.POINTER(_vp)]),
    "bigcn_pipeline_submit": (ctypes.c_int, [_vp, _vp, _vp]),
    "bigcn_pipeline_submit_packed": (ctypes.c_int, [_vp, _vp, _vp, _vp]),
    "bigcn_pipeline_wait": (ctypes.c_int, [_vp]),
    "bigcn_pipeline_close": (ctypes.c_int, [_vp]),
    "bigcn_col_stats": (ctypes.c_int, [_vp, _vp, _i64, _i32, _i64, ctypes.c_float, _vp, _vp]),
    "bigcn_mean_adjacency": (ctypes.c_int, [_vp, _i64, _i64, _vp, _vp, _vp, _vp, _vp, _vp,
                                            ctypes.POINTER(_i64)]),
    "bigcn_sage_layer_forward": (ctypes.c_int, [_vp, ctypes.POINTER(bigcn_graph), ctypes.POINTER(bigcn_layer),
                                                ctypes.POINTER(bigcn_layer), _vp, _vp, _vp, _i64,
                                                ctypes.POINTER(bigcn_layer), _vp, _vp]),
    "bigcn_entropy_bins": (ctypes.c_int, [_vp, _vp, _i64, _i32, _i64, _i32, _vp, _vp, _vp, _vp, _vp]),
    "bigcn_backward_workspace_bytes": (_sz, [_i64, _i32, _i32]),
    "bigcn_layer_backward": (ctypes.c_int, [_vp, ctypes.POINTER(bigcn_graph), ctypes.POINTER(bigcn_layer), _vp, _i64,
                                            _vp, _vp, _vp, _i64, _vp, _i64, _vp, _i64]),
    "bigcn_measure_popc_peak": (ctypes.c_int, [_vp, ctypes.POINTER(ctypes.c_double)]),
    "bigcn_measure_gather_peak": (ctypes.c_int, [_vp, _vp, ctypes.c_int32, ctypes.POINTER(ctypes.c_double)]),
    "bigcn_layer_forward_noalloc": (ctypes.c_int, [_vp, ctypes.POINTER(bigcn_graph), ctypes.POINTER(bigcn_layer),
                                                   _vp, _vp, _vp, _i64, ctypes.POINTER(bigcn_layer), _vp, _vp]),
}

NOALLOC_SCRATCH_BYTES = 8 * 1024 * 1024

_lib = None


def load() -> ctypes.CDLL:
    """Loads libbigcn.so from the package directory (build it with ``python -m
    paper_2210_13149_b200.build`` or ``__graft_entry__.build()``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libbigcn.so is not built (%s): run paper_2210_13149_b200/build.py; "
                               "there is no fallback path" % LIB_PATH)
        lib = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype = res
            fn.argtypes = args
        _lib = lib
    return _lib


class BigcnError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__("bigcn status %d: %s" % (status, message))
        self.status = status


def packed_stride_words(length: int) -> int:
    return int(load().bigcn_packed_stride_words(int(length)))


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


@dataclass
class Graph:
    """Device-resident CSR of A_tilde plus the C struct that points at it."""
    n: int
    nnz: int
    rowptr: torch.Tensor
    colidx: torch.Tensor
    val: torch.Tensor
    dinv: Optional[torch.Tensor]
    c: bigcn_graph


def make_graph(rowptr: torch.Tensor, colidx: torch.Tensor, val: torch.Tensor,
               dinv: Optional[torch.Tensor] = None) -> Graph:
    assert rowptr.dtype == torch.int64 and colidx.dtype == torch.int32 and val.dtype == torch.float32
    n = rowptr.numel() - 1
    nnz = colidx.numel()
    c = bigcn_graph(n, nnz, rowptr.data_ptr(), colidx.data_ptr(), val.data_ptr(),
                    dinv.data_ptr() if dinv is not None else None)
    return Graph(n, nnz, rowptr, colidx, val, dinv, c)


@dataclass
class Layer:
    """Device-resident packed weights of one layer plus the C struct that points at them."""
    d_in: int
    d_out: int
    w_bitsT: torch.Tensor
    alpha: torch.Tensor
    in_shift: Optional[torch.Tensor]
    in_scale: Optional[torch.Tensor]
    c: bigcn_layer


def make_layer(d_in: int, d_out: int, w_bitsT: torch.Tensor, alpha: torch.Tensor,
               in_shift: Optional[torch.Tensor] = None, in_scale: Optional[torch.Tensor] = None) -> Layer:
    c = bigcn_layer(d_in, d_out, w_bitsT.data_ptr(), alpha.data_ptr(),
                    in_shift.data_ptr() if in_shift is not None else None,
                    in_scale.data_ptr() if in_scale is not None else None)
    return Layer(d_in, d_out, w_bitsT, alpha, in_shift, in_scale, c)


def _layer_array(layers: Sequence[Layer]):
    arr = (bigcn_layer * len(layers))()
    for i, l in enumerate(layers):
        arr[i] = l.c
    return arr


def layer_forward_noalloc(graph: "Graph", layer: "Layer", in_bits: torch.Tensor, in_beta: torch.Tensor,
                          h_out: Optional[torch.Tensor] = None, next_layer: Optional["Layer"] = None,
                          next_bits: Optional[torch.Tensor] = None, next_beta: Optional[torch.Tensor] = None,
                          stream: Optional[torch.cuda.Stream] = None) -> int:
    """bigcn_layer_forward_noalloc(): one layer for callers that must not allocate device memory.

    Needs no context and no workspace (the scratch is a fixed array inside the library) and this
    wrapper allocates nothing either: every output tensor is passed in by the caller.  Returns the
    status code (0 = ok; 5 = the problem does not fit the built-in scratch).  Calls must not overlap
    on the GPU: they share the one scratch array."""
    lib = load()
    s = stream if stream is not None else torch.cuda.current_stream()
    return int(lib.bigcn_layer_forward_noalloc(
        ctypes.c_void_p(s.cuda_stream), ctypes.byref(graph.c), ctypes.byref(layer.c), _ptr(in_bits), _ptr(in_beta),
        _ptr(h_out), h_out.stride(0) if h_out is not None else 0,
        ctypes.byref(next_layer.c) if next_layer is not None else None, _ptr(next_bits), _ptr(next_beta)))


class BiGCN:
    """One library context bound to a device and to torch's current stream on it."""

    def __init__(self, device: int = 0, stream: Optional[torch.cuda.Stream] = None):
        self.lib = load()
        if not torch.cuda.is_available():
            raise RuntimeError("no CUDA device: the bigcn library has no CPU path")
        self.device = torch.device("cuda", device)
        with torch.cuda.device(self.device):
            self.stream = stream if stream is not None else torch.cuda.current_stream()
        h = _vp()
        st = self.lib.bigcn_create(ctypes.byref(h), device, ctypes.c_void_p(self.stream.cuda_stream))
        if st != 0:
            raise BigcnError(st, self.lib.bigcn_status_string(st).decode())
        self.h = h
        self.workspace: Optional[torch.Tensor] = None

    def close(self):
        if getattr(self, "h", None):
            self.lib.bigcn_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- helpers
    def _check(self, st: int):
        if st != 0:
            raise BigcnError(st, self.lib.bigcn_last_error(self.h).decode())

    def _empty(self, shape, dtype):
        return torch.empty(shape, dtype=dtype, device=self.device)

    def set_option(self, option: int, value: int):
        self._check(self.lib.bigcn_set_option(self.h, option, value))

    def launch_count(self) -> int:
        return int(self.lib.bigcn_launch_count(self.h))

    def sync_check(self):
        self._check(self.lib.bigcn_sync_check(self.h))

    def workspace_bytes(self, n: int, nnz: int, dims: Sequence[int], host_io: int = 0) -> int:
        arr = (_i32 * len(dims))(*[int(d) for d in dims])
        return int(self.lib.bigcn_workspace_bytes(n, nnz, arr, len(dims) - 1, int(host_io)))

    def ensure_workspace(self, nbytes: int):
        if self.workspace is None or self.workspace.numel() < nbytes:
            self.workspace = None
            self.workspace = torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=self.device)
            self._check(self.lib.bigcn_set_workspace(self.h, _ptr(self.workspace), self.workspace.numel()))

    # -- the ABI calls
    def normalize_adjacency(self, rowptr_A: torch.Tensor, colidx_A: torch.Tensor) -> Graph:
        n = rowptr_A.numel() - 1
        nnz_in = colidx_A.numel()
        self.ensure_workspace(16 * (n // 1024 + 2) + 64)
        rowptr = self._empty(n + 1, torch.int64)
        colidx = self._empty(nnz_in + n, torch.int32)
        val = self._empty(nnz_in + n, torch.float32)
        dinv = self._empty(n, torch.float32)
        nnz = _i64(0)
        self._check(self.lib.bigcn_normalize_adjacency(self.h, n, nnz_in, _ptr(rowptr_A), _ptr(colidx_A),
                                                       _ptr(rowptr), _ptr(colidx), _ptr(val), _ptr(dinv),
                                                       ctypes.byref(nnz)))
        k = int(nnz.value)
        return make_graph(rowptr, colidx[:k], val[:k], dinv)

    def adjacency_from_edges(self, n: int, src: torch.Tensor, dst: torch.Tensor):
        """Canonical CSR pattern of A (rowptr int64, colidx int32) from a raw list of node pairs (device int32)."""
        m = src.numel()
        assert src.dtype == torch.int32 and dst.dtype == torch.int32 and dst.numel() == m
        self.ensure_workspace(int(self.lib.bigcn_edges_workspace_bytes(n, m)))
        rowptr = self._empty(n + 1, torch.int64)
        colidx = self._empty(max(2 * m, 1), torch.int32)
        nnz = _i64(0)
        self._check(self.lib.bigcn_adjacency_from_edges(self.h, n, m, _ptr(src), _ptr(dst), _ptr(rowptr), _ptr(colidx),
                                                        ctypes.byref(nnz)))
        return rowptr, colidx[:int(nnz.value)]

    def pack_features(self, H: torch.Tensor, shift: Optional[torch.Tensor] = None,
                      scale: Optional[torch.Tensor] = None, stride_words: Optional[int] = None):
        n, d = H.shape
        ld = H.stride(0) if n > 1 else d
        assert H.dtype == torch.float32 and (d == 1 or H.stride(1) == 1)
        stride = packed_stride_words(d) if stride_words is None else stride_words
        bits = self._empty((n, stride), torch.int32)
        beta = self._empty(n, torch.float32)
        self._check(self.lib.bigcn_pack_features(self.h, _ptr(H), n, d, ld, _ptr(shift), _ptr(scale),
                                                 _ptr(bits), stride, _ptr(beta)))
        return bits, beta

    def pack_weights(self, W: torch.Tensor):
        d_in, d_out = W.shape
        assert W.dtype == torch.float32 and W.is_contiguous()
        stride = packed_stride_words(d_in)
        bitsT = self._empty((d_out, stride), torch.int32)
        alpha = self._empty(d_out, torch.float32)
        self._check(self.lib.bigcn_pack_weights(self.h, _ptr(W), d_in, d_out, d_out, _ptr(bitsT), stride, _ptr(alpha)))
        return bitsT, alpha

    def layer_forward(self, graph: Graph, layer: Layer, in_bits: torch.Tensor, in_beta: torch.Tensor,
                      want_h: bool = True, next_layer: Optional[Layer] = None, debug: bool = False):
        """Returns dict with h, next_bits, next_beta, dot, zeta (those requested)."""
        n = graph.n
        self.ensure_workspace(self.workspace_bytes(n, graph.nnz, [layer.d_in, layer.d_out]))
        out = {}
        h = self._empty((n, layer.d_out), torch.float32) if want_h else None
        nb = nbeta = None
        if next_layer is not None:
            nb = self._empty((n, packed_stride_words(layer.d_out)), torch.int32)
            nbeta = self._empty(n, torch.float32)
        dot = self._empty((n, layer.d_out), torch.int32) if debug else None
        zeta = self._empty((n, layer.d_out), torch.float32) if debug else None
        self._check(self.lib.bigcn_layer_forward(
            self.h, ctypes.byref(graph.c), ctypes.byref(layer.c), _ptr(in_bits), _ptr(in_beta),
            _ptr(h), layer.d_out, ctypes.byref(next_layer.c) if next_layer is not None else None,
            _ptr(nb), _ptr(nbeta), _ptr(dot), _ptr(zeta)))
        out.update(h=h, next_bits=nb, next_beta=nbeta, dot=dot, zeta=zeta)
        return out

    def _prep_forward(self, graph: Graph, layers: Sequence[Layer], host_io: int = 0):
        dims = [layers[0].d_in] + [l.d_out for l in layers]
        self.ensure_workspace(self.workspace_bytes(graph.n, graph.nnz, dims, host_io))
        return _layer_array(layers), dims

    def forward(self, graph: Graph, layers: Sequence[Layer], X: torch.Tensor,
                logits: Optional[torch.Tensor] = None, stats: bool = False):
        arr, dims = self._prep_forward(graph, layers)
        if logits is None:
            logits = self._empty((graph.n, dims[-1]), torch.float32)
        st = bigcn_stats() if stats else None
        ldx = X.stride(0) if graph.n > 1 else dims[0]
        self._check(self.lib.bigcn_forward(self.h, ctypes.byref(graph.c), arr, len(layers), _ptr(X), ldx,
                                           _ptr(logits), logits.stride(0) if graph.n > 1 else dims[-1],
                                           ctypes.byref(st) if stats else None))
        return (logits, st) if stats else logits

    def forward_packed(self, graph: Graph, layers: Sequence[Layer], x_bits: torch.Tensor, x_beta: torch.Tensor,
                       logits: Optional[torch.Tensor] = None, stats: bool = False):
        arr, dims = self._prep_forward(graph, layers)
        if logits is None:
            logits = self._empty((graph.n, dims[-1]), torch.float32)
        st = bigcn_stats() if stats else None
        self._check(self.lib.bigcn_forward_packed(self.h, ctypes.byref(graph.c), arr, len(layers), _ptr(x_bits),
                                                  _ptr(x_beta), _ptr(logits),
                                                  logits.stride(0) if graph.n > 1 else dims[-1],
                                                  ctypes.byref(st) if stats else None))
        return (logits, st) if stats else logits

    def forward_host(self, graph: Graph, layers: Sequence[Layer], X_host: torch.Tensor,
                     logits_host: torch.Tensor):
        """X_host / logits_host are CPU tensors (pinned for speed); synchronous."""
        arr, dims = self._prep_forward(graph, layers, host_io=True)
        assert X_host.device.type == "cpu" and logits_host.device.type == "cpu"
        assert X_host.is_contiguous() and logits_host.is_contiguous()
        self._check(self.lib.bigcn_forward_host(self.h, ctypes.byref(graph.c), arr, len(layers), _ptr(X_host),
                                                dims[0], _ptr(logits_host), dims[-1]))
        return logits_host

    def open_pipeline(self, graph: Graph, layers: Sequence[Layer], slots: int = 3) -> "Pipeline":
        """Overlapped back-to-back forwards from host buffers (bigcn_pipeline_*)."""
        arr, dims = self._prep_forward(graph, layers, host_io=slots)
        h = _vp()
        self._check(self.lib.bigcn_pipeline_open(self.h, ctypes.byref(graph.c), arr, len(layers), slots, ctypes.byref(h)))
        return Pipeline(self, h, graph, list(layers), dims)

    def layer_backward(self, graph: Graph, layer: Layer, W: torch.Tensor, in_bits: torch.Tensor,
                       in_beta: torch.Tensor, g_out: torch.Tensor, want_g_in: bool = True):
        """Algorithm 1 for one layer: returns (g_in or None, g_w)."""
        n = graph.n
        self.ensure_workspace(int(self.lib.bigcn_backward_workspace_bytes(n, layer.d_in, layer.d_out)))
        g_in = self._empty((n, layer.d_in), torch.float32) if want_g_in else None
        g_w = self._empty((layer.d_in, layer.d_out), torch.float32)
        self._check(self.lib.bigcn_layer_backward(
            self.h, ctypes.byref(graph.c), ctypes.byref(layer.c), _ptr(W), W.stride(0) if layer.d_in > 1 else layer.d_out,
            _ptr(in_bits), _ptr(in_beta), _ptr(g_out), g_out.stride(0) if n > 1 else layer.d_out,
            _ptr(g_in), layer.d_in, _ptr(g_w), layer.d_out))
        return g_in, g_w

    def entropy_bins(self, H: torch.Tensor, n_bins: int):
        """Binning entropy estimate (Sec. 6.2): dict of col_min, col_max, counts [d x n_bins], entropy [d] (bits), total."""
        n, d = H.shape
        self.ensure_workspace(8 * d)
        out = dict(col_min=self._empty(d, torch.float32), col_max=self._empty(d, torch.float32),
                   counts=self._empty((d, n_bins), torch.int32), entropy=self._empty(d, torch.float64),
                   total=self._empty(1, torch.float64))
        self._check(self.lib.bigcn_entropy_bins(self.h, _ptr(H), n, d, H.stride(0) if n > 1 else d, n_bins,
                                                _ptr(out["col_min"]), _ptr(out["col_max"]), _ptr(out["counts"]),
                                                _ptr(out["entropy"]), _ptr(out["total"])))
        return out

    def col_stats(self, H: torch.Tensor, eps: float = 1e-5):
        n, d = H.shape
        self.ensure_workspace(16 * d * 1024)
        shift = self._empty(d, torch.float32)
        scale = self._empty(d, torch.float32)
        self._check(self.lib.bigcn_col_stats(self.h, _ptr(H), n, d, H.stride(0) if n > 1 else d, eps,
                                             _ptr(shift), _ptr(scale)))
        return shift, scale

    def mean_adjacency(self, rowptr_A: torch.Tensor, colidx_A: torch.Tensor) -> Graph:
        n = rowptr_A.numel() - 1
        nnz_in = colidx_A.numel()
        self.ensure_workspace(16 * (n // 1024 + 2) + 64)
        rowptr = self._empty(n + 1, torch.int64)
        colidx = self._empty(max(nnz_in, 1), torch.int32)
        val = self._empty(max(nnz_in, 1), torch.float32)
        inv_deg = self._empty(n, torch.float32)
        nnz = _i64(0)
        self._check(self.lib.bigcn_mean_adjacency(self.h, n, nnz_in, _ptr(rowptr_A), _ptr(colidx_A),
                                                  _ptr(rowptr), _ptr(colidx), _ptr(val), _ptr(inv_deg),
                                                  ctypes.byref(nnz)))
        k = int(nnz.value)
        return make_graph(rowptr, colidx[:k], val[:k], inv_deg)

    def sage_layer_forward(self, mean_graph: Graph, self_layer: Layer, nbr_layer: Layer, in_bits: torch.Tensor,
                           in_beta: torch.Tensor, want_h: bool = True, next_layer: Optional[Layer] = None):
        """Returns dict with h, next_bits, next_beta (those requested)."""
        n = mean_graph.n
        self.ensure_workspace(2 * self.workspace_bytes(n, mean_graph.nnz, [self_layer.d_in, self_layer.d_out]))
        d_out = self_layer.d_out
        h = self._empty((n, d_out), torch.float32) if want_h else None
        nb = nbeta = None
        if next_layer is not None:
            nb = self._empty((n, packed_stride_words(d_out)), torch.int32)
            nbeta = self._empty(n, torch.float32)
        self._check(self.lib.bigcn_sage_layer_forward(
            self.h, ctypes.byref(mean_graph.c), ctypes.byref(self_layer.c), ctypes.byref(nbr_layer.c),
            _ptr(in_bits), _ptr(in_beta), _ptr(h), d_out,
            ctypes.byref(next_layer.c) if next_layer is not None else None, _ptr(nb), _ptr(nbeta)))
        return {"h": h, "next_bits": nb, "next_beta": nbeta}

    def measure_popc_peak(self) -> float:
        """32-bit XOR + bit-count + add steps per second of this GPU (register-only probe)."""
        self.ensure_workspace(2 << 20)
        out = ctypes.c_double(0.0)
        self._check(self.lib.bigcn_measure_popc_peak(self.h, ctypes.byref(out)))
        return float(out.value)

    def measure_gather_peak(self, G, row_bytes: int) -> float:
        """Milliseconds the memory system alone needs to read, for every stored entry of G, the row of
        `row_bytes` bytes its column index names (the aggregation's gather without any arithmetic)."""
        self.ensure_workspace(G.n * row_bytes + (1 << 20))
        out = ctypes.c_double(0.0)
        self._check(self.lib.bigcn_measure_gather_peak(self.h, ctypes.byref(G.c), int(row_bytes), ctypes.byref(out)))
        return float(out.value)

    # -- convenience built only from the calls above
    def prepare_layers(self, weights: Sequence[torch.Tensor], shifts=None, scales=None) -> List[Layer]:
        layers = []
        for l, W in enumerate(weights):
            bitsT, alpha = self.pack_weights(W)
            sh = shifts[l] if shifts is not None else None
            sc = scales[l] if scales is not None else None
            layers.append(make_layer(W.shape[0], W.shape[1], bitsT, alpha, sh, sc))
        return layers


class Pipeline:
    """bigcn_pipeline_*: submit() enqueues a step from pinned host tensors, wait() blocks for the oldest one."""

    def __init__(self, ctx: BiGCN, handle, graph: Graph, layers: List[Layer], dims: List[int]):
        self.ctx, self.h, self.graph, self.layers, self.dims = ctx, handle, graph, layers, dims
        self._held = []                     # host tensors of outstanding steps stay referenced

    def submit(self, X_host: torch.Tensor, logits_host: torch.Tensor):
        assert X_host.device.type == "cpu" and logits_host.device.type == "cpu"
        assert X_host.is_contiguous() and logits_host.is_contiguous()
        assert tuple(X_host.shape) == (self.graph.n, self.dims[0]) and X_host.dtype == torch.float32
        assert tuple(logits_host.shape) == (self.graph.n, self.dims[-1]) and logits_host.dtype == torch.float32
        self.ctx._check(self.ctx.lib.bigcn_pipeline_submit(self.h, _ptr(X_host), _ptr(logits_host)))
        self._held.append((X_host, logits_host))

    def submit_packed(self, bits_host: torch.Tensor, beta_host: torch.Tensor, logits_host: torch.Tensor):
        """A step from an already binary input (packed sign bits and beta, host tensors)."""
        n = self.graph.n
        assert bits_host.device.type == "cpu" and beta_host.device.type == "cpu" and logits_host.device.type == "cpu"
        assert bits_host.is_contiguous() and beta_host.is_contiguous() and logits_host.is_contiguous()
        assert tuple(bits_host.shape) == (n, packed_stride_words(self.dims[0])) and bits_host.dtype == torch.int32
        assert tuple(beta_host.shape) == (n,) and beta_host.dtype == torch.float32
        assert tuple(logits_host.shape) == (n, self.dims[-1]) and logits_host.dtype == torch.float32
        self.ctx._check(self.ctx.lib.bigcn_pipeline_submit_packed(self.h, _ptr(bits_host), _ptr(beta_host), _ptr(logits_host)))
        self._held.append(((bits_host, beta_host), logits_host))

    def wait(self) -> Optional[torch.Tensor]:
        self.ctx._check(self.ctx.lib.bigcn_pipeline_wait(self.h))
        return self._held.pop(0)[1] if self._held else None

    def close(self):
        if getattr(self, "h", None):
            self.ctx.lib.bigcn_pipeline_close(self.h)
            self.h = None
            self._held = []

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

"""CPU oracle of the binarized Bi-GCN forward path (Bi-GCN, Sec. 3, 4.1, 4.2, 4.4, 5).

TEST INFRASTRUCTURE ONLY: a plain restatement of the paper's definitions used to
check the CUDA library.  Nothing here is shared with, imported by, or imports
the CUDA path.  The arithmetic lives in ``bigcn_oracle.c`` (one loop per
definition, double accumulation); this module only marshals numpy arrays into
it and strings the steps together in the paper's order.

Pinned by the ``-m "not gpu"`` tests (brute force over sign vectors, dense +-1
float products, dense N x N adjacency products, hand-worked star/path graphs,
the fp32 GCN layer on +-1 inputs, Table 1 of the paper).  The value of a full
forward on the paper's own datasets is "parity unpinned": the paper prints no
numerical example and the datasets are not available.
"""
from __future__ import annotations

import ctypes
import os
import platform
import subprocess
from dataclasses import dataclass
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "bigcn_oracle.c")
_LIB = os.path.join(_HERE, "libbigcn_oracle.so")

_c_i64 = ctypes.c_int64
_c_i32 = ctypes.c_int32
_c_f64 = ctypes.c_double
_vp = ctypes.c_void_p


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP over rows, no FMA contraction)."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + ".%d.tmp" % os.getpid()
    cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
           "-fno-fast-math", "-o", tmp, _SRC, "-lm"]
    if platform.machine() in ("x86_64", "AMD64"):
        cmd.insert(1, "-mpopcnt")
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        L.oracle_num_threads.restype = ctypes.c_int
        L.oracle_set_num_threads.argtypes = [ctypes.c_int]
        L.oracle_normalize_adjacency.restype = _c_i64
        L.oracle_normalize_adjacency.argtypes = [_c_i64, _c_i64, _vp, _vp, _vp, _vp, _vp, _vp]
        L.oracle_col_stats.argtypes = [_vp, _c_i64, _c_i32, _c_i64, _c_f64, _vp, _vp]
        L.oracle_binarize_rows.argtypes = [_vp, _c_i64, _c_i32, _c_i64, _vp, _vp, _vp, _vp]
        L.oracle_binarize_cols.argtypes = [_vp, _c_i32, _c_i32, _c_i64, _vp, _vp]
        L.oracle_pack_rows.argtypes = [_vp, _c_i64, _c_i32, _vp, _c_i64]
        L.oracle_pack_cols.argtypes = [_vp, _c_i32, _c_i32, _vp, _c_i64]
        L.oracle_unpack_rows.argtypes = [_vp, _c_i64, _c_i64, _c_i32, _vp]
        L.oracle_dot_pm1.argtypes = [_vp, _vp, _c_i64, _c_i32, _c_i32, _vp]
        L.oracle_dot_popc.argtypes = [_vp, _c_i64, _vp, _c_i64, _c_i64, _c_i32, _c_i32, _vp]
        L.oracle_rescale.argtypes = [_vp, _vp, _vp, _c_i64, _c_i32, _vp, _c_i64]
        L.oracle_spmm.argtypes = [_c_i64, _vp, _vp, _vp, _vp, _c_i32, _c_i64, _vp, _c_i64]
        L.oracle_cost_model.argtypes = [_c_f64, _c_f64, _vp, _c_i32, _vp]
        L.oracle_mean_adjacency.restype = _c_i64
        L.oracle_mean_adjacency.argtypes = [_c_i64, _c_i64, _vp, _vp, _vp, _vp, _vp, _vp]
        L.oracle_spmm_add.argtypes = [_c_i64, _vp, _vp, _vp, _vp, _c_i32, _c_i64, _vp, _c_i64, _vp, _c_i64]
        L.oracle_entropy_bins.argtypes = [_vp, _c_i64, _c_i32, _c_i64, _c_i32, _vp, _vp, _vp, _vp]
        L.oracle_entropy_bins.restype = _c_f64
        L.oracle_layer_backward.argtypes = [_c_i64, _vp, _vp, _vp, _c_i32, _c_i32, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
        _lib = L
    return _lib


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def set_num_threads(t: int) -> None:
    lib().oracle_set_num_threads(int(t))


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(_vp)


def _arr(a, dtype) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=dtype)


def stride_words(d: int) -> int:
    """Words per packed row: ceil(d / 32) rounded up to a multiple of 4 (16 bytes)."""
    kw = (int(d) + 31) // 32
    return (kw + 3) // 4 * 4


# --------------------------------------------------------------------------- steps

@dataclass
class Graph:
    """CSR of A_tilde = D_hat^-1/2 (A + I) D_hat^-1/2 (Eq. 1)."""
    n: int
    rowptr: np.ndarray   # int64 [n+1]
    colidx: np.ndarray   # int32 [nnz], ascending within a row, diagonal included
    val: np.ndarray      # float32 [nnz]
    dinv: np.ndarray     # float32 [n]

    @property
    def nnz(self) -> int:
        return int(self.rowptr[-1])


def normalize_adjacency(n: int, src, dst) -> Graph:
    src = _arr(src, np.int32)
    dst = _arr(dst, np.int32)
    m = int(src.shape[0])
    assert dst.shape[0] == m
    rowptr = np.zeros(n + 1, dtype=np.int64)
    colidx = np.zeros(2 * m + n, dtype=np.int32)
    val = np.zeros(2 * m + n, dtype=np.float32)
    dinv = np.zeros(n, dtype=np.float32)
    nnz = lib().oracle_normalize_adjacency(n, m, _p(src), _p(dst), _p(rowptr), _p(colidx),
                                           _p(val), _p(dinv))
    if nnz < 0:
        raise ValueError("edge list has a node id outside [0, n)")
    return Graph(n, rowptr, colidx[:nnz].copy(), val[:nnz].copy(), dinv)


def col_stats(H: np.ndarray, eps: float = 1e-5):
    H = _arr(H, np.float32)
    n, d = H.shape
    shift = np.zeros(d, np.float32)
    scale = np.zeros(d, np.float32)
    lib().oracle_col_stats(_p(H), n, d, d, float(eps), _p(shift), _p(scale))
    return shift, scale


def binarize_rows(H: np.ndarray, shift=None, scale=None):
    """F (+-1 int8, n x d) and beta (float32, n) of Sec. 4.2.2."""
    H = _arr(H, np.float32)
    n, d = H.shape
    if shift is not None:
        shift = _arr(shift, np.float32)
        scale = _arr(scale, np.float32)
        assert shift.shape == (d,) and scale.shape == (d,)
    F = np.zeros((n, d), np.int8)
    beta = np.zeros(n, np.float32)
    lib().oracle_binarize_rows(_p(H), n, d, d, _p(shift), _p(scale), _p(F), _p(beta))
    return F, beta


def binarize_cols(W: np.ndarray):
    """B (+-1 int8, d_in x d_out) and alpha (float32, d_out) of Sec. 4.2.1."""
    W = _arr(W, np.float32)
    d_in, d_out = W.shape
    B = np.zeros((d_in, d_out), np.int8)
    alpha = np.zeros(d_out, np.float32)
    lib().oracle_binarize_cols(_p(W), d_in, d_out, d_out, _p(B), _p(alpha))
    return B, alpha


def pack_rows(F: np.ndarray, stride: Optional[int] = None) -> np.ndarray:
    F = _arr(F, np.int8)
    n, d = F.shape
    stride = stride_words(d) if stride is None else int(stride)
    bits = np.zeros((n, stride), np.uint32)
    lib().oracle_pack_rows(_p(F), n, d, _p(bits), stride)
    return bits


def pack_cols(B: np.ndarray, stride: Optional[int] = None) -> np.ndarray:
    B = _arr(B, np.int8)
    d_in, d_out = B.shape
    stride = stride_words(d_in) if stride is None else int(stride)
    bitsT = np.zeros((d_out, stride), np.uint32)
    lib().oracle_pack_cols(_p(B), d_in, d_out, _p(bitsT), stride)
    return bitsT


def unpack_rows(bits: np.ndarray, d: int) -> np.ndarray:
    bits = _arr(bits, np.uint32)
    n, stride = bits.shape
    F = np.zeros((n, d), np.int8)
    lib().oracle_unpack_rows(_p(bits), stride, n, d, _p(F))
    return F


def dot_pm1(F: np.ndarray, B: np.ndarray) -> np.ndarray:
    F = _arr(F, np.int8)
    B = _arr(B, np.int8)
    n, d_in = F.shape
    assert B.shape[0] == d_in
    d_out = B.shape[1]
    dot = np.zeros((n, d_out), np.int32)
    lib().oracle_dot_pm1(_p(F), _p(B), n, d_in, d_out, _p(dot))
    return dot


def dot_popc(bits: np.ndarray, bitsT: np.ndarray, d_in: int) -> np.ndarray:
    bits = _arr(bits, np.uint32)
    bitsT = _arr(bitsT, np.uint32)
    n, sa = bits.shape
    d_out, sb = bitsT.shape
    dot = np.zeros((n, d_out), np.int32)
    lib().oracle_dot_popc(_p(bits), sa, _p(bitsT), sb, n, d_in, d_out, _p(dot))
    return dot


def rescale(dot: np.ndarray, beta: np.ndarray, alpha: np.ndarray) -> np.ndarray:
    dot = _arr(dot, np.int32)
    beta = _arr(beta, np.float32)
    alpha = _arr(alpha, np.float32)
    n, d_out = dot.shape
    zeta = np.zeros((n, d_out), np.float32)
    lib().oracle_rescale(_p(dot), _p(beta), _p(alpha), n, d_out, _p(zeta), d_out)
    return zeta


def spmm(g: Graph, zeta: np.ndarray, row_begin: int = 0, row_end: Optional[int] = None) -> np.ndarray:
    """Rows [row_begin, row_end) of A_tilde @ zeta."""
    zeta = _arr(zeta, np.float32)
    assert zeta.shape[0] == g.n
    d_out = zeta.shape[1]
    row_end = g.n if row_end is None else int(row_end)
    rows = row_end - row_begin
    out = np.zeros((rows, d_out), np.float32)
    rp = g.rowptr[row_begin:row_end + 1]
    lib().oracle_spmm(rows, _p(rp), _p(g.colidx), _p(g.val), _p(zeta), d_out, d_out, _p(out), d_out)
    return out


def cost_model(n: float, e: float, dims: Sequence[int]) -> dict:
    dims_a = _arr(dims, np.int32)
    out = np.zeros(6, np.float64)
    lib().oracle_cost_model(float(n), float(e), _p(dims_a), len(dims) - 1, _p(out))
    return {"ops_gcn": out[0], "ops_bigcn": out[1], "model_bytes_gcn": out[2],
            "model_bytes_bigcn": out[3], "data_bytes_gcn": out[4], "data_bytes_bigcn": out[5]}


# --------------------------------------------------------------------------- the layer and the network

@dataclass
class Layer:
    """One binarized graph-convolution layer: fp32 weights W (d_in x d_out) and the optional
    inference-mode batch-norm constants of its input (Sec. 4.4)."""
    W: np.ndarray
    in_shift: Optional[np.ndarray] = None
    in_scale: Optional[np.ndarray] = None


@dataclass
class LayerTrace:
    F: np.ndarray
    beta: np.ndarray
    bits: np.ndarray
    bitsT: np.ndarray
    alpha: np.ndarray
    dot: np.ndarray
    zeta: np.ndarray
    H_out: np.ndarray


def layer_forward(g: Graph, layer: Layer, H: np.ndarray, use_pm1: bool = False) -> LayerTrace:
    """Sec. 4.2 in the paper's order: (BN) -> sign / beta -> sign / alpha -> F (*) B by XNOR and bit
    count -> beta_i alpha_j rescale -> A_tilde zeta.  No bias, no ReLU (Sec. 4.2.2)."""
    d_in = layer.W.shape[0]
    F, beta = binarize_rows(H, layer.in_shift, layer.in_scale)
    B, alpha = binarize_cols(layer.W)
    bits = pack_rows(F)
    bitsT = pack_cols(B)
    dot = dot_pm1(F, B) if use_pm1 else dot_popc(bits, bitsT, d_in)
    zeta = rescale(dot, beta, alpha)
    H_out = spmm(g, zeta)
    return LayerTrace(F, beta, bits, bitsT, alpha, dot, zeta, H_out)


def layer_forward_packed(g: Graph, layer: Layer, bits: np.ndarray, beta: np.ndarray) -> LayerTrace:
    """The same layer from an input that is already binary (Sec. 5.2: packed signs F and one
    scalar beta_i per node): sign / alpha of the weights -> F (*) B -> rescale -> A_tilde zeta.
    The layer's batch-norm constants are not used: they act before the binarization."""
    d_in = layer.W.shape[0]
    bits = _arr(bits, np.uint32)
    beta = _arr(beta, np.float32)
    F = unpack_rows(bits, d_in)
    B, alpha = binarize_cols(layer.W)
    bitsT = pack_cols(B)
    dot = dot_popc(pack_rows(F), bitsT, d_in)
    zeta = rescale(dot, beta, alpha)
    H_out = spmm(g, zeta)
    return LayerTrace(F, beta, bits, bitsT, alpha, dot, zeta, H_out)


def forward(g: Graph, layers: List[Layer], X: np.ndarray, keep_trace: bool = True):
    """L stacked layers, H^(0) = X; the last layer's output is the logits (Sec. 3.2)."""
    H = X
    traces = []
    for layer in layers:
        t = layer_forward(g, layer, H)
        H = t.H_out
        if keep_trace:
            traces.append(t)
        else:
            del t
    return H, traces


def calibrate_bn(g: Graph, weights: List[np.ndarray], X: np.ndarray, bn_layers: Sequence[bool],
                 eps: float = 1e-5) -> List[Layer]:
    """Freeze inference-mode batch-norm constants (Sec. 4.4, Sec. 7 setups): for every layer
    flagged in ``bn_layers`` take the column statistics of that layer's input as the oracle
    itself produces it, layer after layer."""
    layers: List[Layer] = []
    H = X
    for l, W in enumerate(weights):
        if bn_layers[l]:
            shift, scale = col_stats(H, eps)
            layer = Layer(W, shift, scale)
        else:
            layer = Layer(W)
        layers.append(layer)
        if l + 1 < len(weights):
            H = layer_forward(g, layer, H).H_out
    return layers


# --------------------------------------------------------------------------- Bi-GraphSAGE (Sec. 4.4.2)

def mean_adjacency(n: int, src, dst) -> Graph:
    """CSR of the mean aggregator: row i holds 1/|N_i| on its distinct neighbours (no self-loop).
    The returned Graph's ``dinv`` field holds 1/|N_i| (0 for isolated nodes)."""
    src = _arr(src, np.int32)
    dst = _arr(dst, np.int32)
    m = int(src.shape[0])
    rowptr = np.zeros(n + 1, dtype=np.int64)
    colidx = np.zeros(max(2 * m, 1), dtype=np.int32)
    val = np.zeros(max(2 * m, 1), dtype=np.float32)
    inv_deg = np.zeros(n, dtype=np.float32)
    nnz = lib().oracle_mean_adjacency(n, m, _p(src), _p(dst), _p(rowptr), _p(colidx), _p(val), _p(inv_deg))
    if nnz < 0:
        raise ValueError("edge list has a node id outside [0, n)")
    return Graph(n, rowptr, colidx[:nnz].copy(), val[:nnz].copy(), inv_deg)


def spmm_add(g: Graph, z: np.ndarray, self_term: Optional[np.ndarray]) -> np.ndarray:
    """self_term + g @ z, both terms added in double, rounded once."""
    z = _arr(z, np.float32)
    d_out = z.shape[1]
    if self_term is not None:
        self_term = _arr(self_term, np.float32)
        assert self_term.shape == (g.n, d_out)
    out = np.zeros((g.n, d_out), np.float32)
    lib().oracle_spmm_add(g.n, _p(g.rowptr), _p(g.colidx), _p(g.val), _p(z), d_out, d_out,
                          _p(self_term), d_out, _p(out), d_out)
    return out


@dataclass
class SageLayer:
    """One binarized GraphSAGE layer (mean aggregator): weights of the node itself and of its
    neighbours, and the optional batch-norm constants of the layer input."""
    W_self: np.ndarray
    W_nbr: np.ndarray
    in_shift: Optional[np.ndarray] = None
    in_scale: Optional[np.ndarray] = None


@dataclass
class SageTrace:
    F: np.ndarray
    beta: np.ndarray
    bits: np.ndarray
    bitsT_self: np.ndarray
    alpha_self: np.ndarray
    bitsT_nbr: np.ndarray
    alpha_nbr: np.ndarray
    zeta_self: np.ndarray
    zeta_nbr: np.ndarray
    H_out: np.ndarray


def sage_layer_forward(g_mean: Graph, layer: SageLayer, H: np.ndarray) -> SageTrace:
    """Eq. "bisage-conv": h_i' = W_theta (*) h_i + (1/|N_i|) sum_j W_n (*) h_j, both products by XNOR and
    bit count on the same binarized input, no activation."""
    d_in = layer.W_self.shape[0]
    F, beta = binarize_rows(H, layer.in_shift, layer.in_scale)
    bits = pack_rows(F)
    Bs, a_s = binarize_cols(layer.W_self)
    Bn, a_n = binarize_cols(layer.W_nbr)
    bT_s, bT_n = pack_cols(Bs), pack_cols(Bn)
    z_s = rescale(dot_popc(bits, bT_s, d_in), beta, a_s)
    z_n = rescale(dot_popc(bits, bT_n, d_in), beta, a_n)
    H_out = spmm_add(g_mean, z_n, z_s)
    return SageTrace(F, beta, bits, bT_s, a_s, bT_n, a_n, z_s, z_n, H_out)


@dataclass
class EntropyEstimate:
    """Binning estimate of Sec. 6.2: per-neuron range, interval counts, entropies in bits, and their sum."""
    col_min: np.ndarray      # [d] float32
    col_max: np.ndarray      # [d] float32
    counts: np.ndarray       # [d, M] int64
    entropy: np.ndarray      # [d] float64, bits
    total: float             # H_ind = sum of the per-neuron entropies


def entropy_bins(H: np.ndarray, n_bins: int) -> EntropyEstimate:
    """H_hat(h_i) = -sum_m p log2 p over M equal-width intervals of each column's own range (Sec. 6.2)."""
    H = _arr(H, np.float32)
    n, d = H.shape
    lo = np.empty(d, np.float32)
    hi = np.empty(d, np.float32)
    counts = np.empty((d, n_bins), np.int64)
    ent = np.empty(d, np.float64)
    total = lib().oracle_entropy_bins(_p(H), n, d, H.shape[1], n_bins, _p(lo), _p(hi), _p(counts), _p(ent))
    return EntropyEstimate(lo, hi, counts, ent, float(total))


@dataclass
class BackwardTrace:
    """Algorithm 1 for one layer: the three gradients of step 1, then Eq. bp-H and Eq. bp-W."""
    G_zeta: np.ndarray       # [n, d_out]   A_tilde^T G'
    G_Wt: np.ndarray         # [d_in, d_out] gradient of the binarized weights W~
    G_Ht: np.ndarray         # [n, d_in]    gradient of the binarized input H~
    G_H: np.ndarray          # [n, d_in]    Eq. bp-H
    G_W: np.ndarray          # [d_in, d_out] Eq. bp-W


def layer_backward(g: Graph, W: np.ndarray, F: np.ndarray, beta: np.ndarray, G_out: np.ndarray) -> BackwardTrace:
    """Back-propagation through H' = A_tilde ((beta F)(alpha B)) with B, alpha from W (Algorithm 1, Sec. 4.3).
    F is the +-1 input of the forward pass and beta its row scales."""
    W = _arr(W, np.float32)
    d_in, d_out = W.shape
    Bm, alpha = binarize_cols(W)
    F = _arr(F, np.int8)
    beta = _arr(beta, np.float32)
    G_out = _arr(G_out, np.float32)
    n = g.n
    assert F.shape == (n, d_in) and G_out.shape == (n, d_out)
    out = BackwardTrace(np.empty((n, d_out), np.float32), np.empty((d_in, d_out), np.float32),
                        np.empty((n, d_in), np.float32), np.empty((n, d_in), np.float32),
                        np.empty((d_in, d_out), np.float32))
    lib().oracle_layer_backward(n, _p(g.rowptr), _p(g.colidx), _p(g.val), d_in, d_out, _p(F), _p(beta), _p(Bm), _p(alpha),
                                _p(W), _p(G_out), _p(out.G_zeta), _p(out.G_Wt), _p(out.G_Ht), _p(out.G_H), _p(out.G_W))
    return out

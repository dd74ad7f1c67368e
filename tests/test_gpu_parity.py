"""GPU parity: every step of the CUDA path against the CPU oracle, through the C ABI.

Packed bits and integer dot products must match exactly; fp32 outputs within
|gpu - oracle| <= 1e-4 + 1e-5 |oracle| when the layer is fed the oracle's own input.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2210_13149_b200 import synth
from parity_util import (ATOL, RTOL, assert_close, bits_from_dev, bits_to_dev, dev, device_graph,
                         device_layers_from_oracle, end_to_end_with_flip_accounting, flip_report, oracle_run)

pytestmark = pytest.mark.gpu

FORMATS = [1, 2, 3, 4, 5]    # fp32 zeta; integer dots as int16 / int8 (d_in <= 127) / fp16 (d_in <= 2048) / half-dot bytes (128 <= d_in <= 256)


@pytest.fixture(scope="module")
def B():
    from paper_2210_13149_b200 import binding
    return binding


@pytest.fixture()
def ctx(B):
    c = B.BiGCN(0)
    yield c
    c.sync_check()
    c.close()


def small_graph(n, e_dir, seed):
    rp, ci = synth.power_law_graph(n, e_dir, seed)
    src, dst = synth.edge_list(rp, ci)
    return rp, ci, oracle.normalize_adjacency(n, src, dst)


# --------------------------------------------------------------------------- set-up step

@pytest.mark.parametrize("n,e,seed", [(1, 0, 1), (7, 0, 2), (50, 200, 3), (2708, 10556, 1001), (5000, 400000, 5)])
def test_normalize_adjacency_is_bit_exact(ctx, n, e, seed):
    rp, ci, g = small_graph(n, e, seed)
    got = ctx.normalize_adjacency(rp.cuda(), ci.cuda())
    assert got.nnz == g.nnz
    assert np.array_equal(got.rowptr.cpu().numpy(), g.rowptr)
    assert np.array_equal(got.colidx.cpu().numpy(), g.colidx)
    assert np.array_equal(got.dinv.cpu().numpy(), g.dinv)
    assert np.array_equal(got.val.cpu().numpy(), g.val)


@pytest.mark.parametrize("n,m,seed", [(1, 0, 1), (5, 0, 2), (2, 7, 3), (60, 500, 4), (3000, 40000, 5), (200000, 1500000, 6)])
def test_adjacency_from_a_raw_edge_list(ctx, B, n, m, seed):
    """The set-up from node pairs as a data set lists them -- one direction or both, repeated, some joining a node to
    itself, many nodes isolated -- followed by the normalisation: structure and values bit for bit what the oracle
    builds from the same list (Sec. 3.1; the oracle symmetrises, de-duplicates and drops self pairs itself)."""
    rng = np.random.default_rng(seed)
    hi = max(n // 2, 1)                                              # the upper half of the ids stays isolated
    src = rng.integers(0, hi, m).astype(np.int32)
    dst = rng.integers(0, hi, m).astype(np.int32)
    if m > 10:
        src[: m // 5], dst[: m // 5] = dst[m // 5: 2 * (m // 5)].copy(), src[m // 5: 2 * (m // 5)].copy()   # reversed copies
        src[-(m // 10):] = src[: m // 10]                            # exact repeats
        dst[-(m // 10):] = dst[: m // 10]
    g = oracle.normalize_adjacency(n, src, dst)
    rp, ci = ctx.adjacency_from_edges(n, dev(src), dev(dst))
    # the pattern of A: the oracle's A_hat without its diagonal
    keep = g.colidx != np.repeat(np.arange(n), np.diff(g.rowptr))
    assert np.array_equal(ci.cpu().numpy(), g.colidx[keep])
    assert np.array_equal(rp.cpu().numpy(), g.rowptr - np.arange(n + 1))
    got = ctx.normalize_adjacency(rp, ci)
    assert got.nnz == g.nnz
    assert np.array_equal(got.rowptr.cpu().numpy(), g.rowptr)
    assert np.array_equal(got.colidx.cpu().numpy(), g.colidx)
    assert np.array_equal(got.val.cpu().numpy(), g.val)
    assert np.array_equal(got.dinv.cpu().numpy(), g.dinv)


def test_adjacency_from_edges_rejects_ids_out_of_range(ctx, B):
    src = dev(np.array([0, 1, 5], np.int32))
    dst = dev(np.array([1, 2, 0], np.int32))
    with pytest.raises(B.BigcnError) as e:
        ctx.adjacency_from_edges(5, src, dst)                        # node 5 of 5
    assert e.value.status == 4                                       # BIGCN_ERR_GRAPH
    with pytest.raises(B.BigcnError) as e:
        ctx.adjacency_from_edges(5, dev(np.array([-1], np.int32)), dev(np.array([0], np.int32)))
    assert e.value.status == 4
    rp, ci = ctx.adjacency_from_edges(6, src, dst)                   # fine with one more node
    assert rp.cpu().tolist() == [0, 2, 4, 5, 5, 5, 6] and ci.cpu().tolist() == [1, 5, 0, 2, 1, 0]


def test_normalize_adjacency_drops_input_diagonal(ctx):
    # path 0-1-2 with self-loops already present on 0 and 2
    rp = torch.tensor([0, 2, 4, 6], dtype=torch.int64)
    ci = torch.tensor([0, 1, 0, 2, 1, 2], dtype=torch.int32)
    g = oracle.normalize_adjacency(3, np.array([0, 1], np.int32), np.array([1, 2], np.int32))
    got = ctx.normalize_adjacency(rp.cuda(), ci.cuda())
    assert np.array_equal(got.colidx.cpu().numpy(), g.colidx)
    assert np.array_equal(got.val.cpu().numpy(), g.val)


@pytest.mark.parametrize("rp,ci", [
    ([0, 1, 1], [1]),                 # (0,1) without (1,0)
    ([0, 2, 3, 4], [2, 1, 0, 0]),     # columns not ascending
    ([0, 1, 2], [1, 5]),              # column out of range
    ([0, 2, 1], [1, 0]),              # rowptr not monotone
])
def test_normalize_adjacency_rejects_malformed_input(ctx, B, rp, ci):
    with pytest.raises(B.BigcnError) as e:
        ctx.normalize_adjacency(torch.tensor(rp, dtype=torch.int64).cuda(), torch.tensor(ci, dtype=torch.int32).cuda())
    assert e.value.status == 4
    ctx.sync_check()                  # the context stays usable


# --------------------------------------------------------------------------- binarize + pack

@pytest.mark.parametrize("n,d", [(1, 1), (5, 31), (9, 32), (13, 33), (300, 100), (77, 602), (40, 1433), (11, 3703), (1000, 256),
                                 (77, 600), (33, 132), (19, 4), (3000, 1436)])   # row lengths that are multiples of 4 take the 16-byte-load kernel
@pytest.mark.parametrize("norm", [False, True])
def test_pack_features(ctx, n, d, norm):
    rng = np.random.default_rng(n * 7919 + d)
    H = rng.standard_normal((n, d)).astype(np.float32)
    H[rng.random((n, d)) < 0.2] = 0.0
    shift = scale = None
    if norm:
        shift, scale = oracle.col_stats(H)
    F, beta = oracle.binarize_rows(H, shift, scale)
    bits = oracle.pack_rows(F)
    gb, gbeta = ctx.pack_features(dev(H), dev(shift) if norm else None, dev(scale) if norm else None)
    assert np.array_equal(bits_from_dev(gb), bits)
    np.testing.assert_allclose(gbeta.cpu().numpy(), beta, rtol=2e-6, atol=1e-30)


def test_pack_features_strided_input_and_wide_output(ctx):
    rng = np.random.default_rng(5)
    n, d, ld = 33, 70, 96
    buf = rng.standard_normal((n, ld)).astype(np.float32)
    H = buf[:, :d]
    F, beta = oracle.binarize_rows(np.ascontiguousarray(H))
    bits = oracle.pack_rows(F, stride=8)
    gb, gbeta = ctx.pack_features(dev(buf)[:, :d], stride_words=8)
    assert np.array_equal(bits_from_dev(gb), bits)
    np.testing.assert_allclose(gbeta.cpu().numpy(), beta, rtol=2e-6)


def test_pack_features_sign_convention(ctx):
    tiny = np.float32(1e-45)
    H = np.array([[0.0, -0.0, tiny, -tiny, 1.0, -1.0, np.inf, -np.inf, np.nan]], np.float32)
    F, _ = oracle.binarize_rows(H)
    gb, _ = ctx.pack_features(dev(H))
    assert np.array_equal(bits_from_dev(gb), oracle.pack_rows(F))
    assert bits_from_dev(gb)[0, 0] == 0b001010111


@pytest.mark.parametrize("d_in,d_out", [(1, 1), (33, 7), (100, 256), (602, 256), (1433, 64), (3703, 64), (256, 47), (64, 3)])
def test_pack_weights(ctx, d_in, d_out):
    rng = np.random.default_rng(d_in * 31 + d_out)
    W = (rng.standard_normal((d_in, d_out)) * d_in ** -0.5).astype(np.float32)
    W[rng.random((d_in, d_out)) < 0.05] = 0.0
    Bm, alpha = oracle.binarize_cols(W)
    bitsT = oracle.pack_cols(Bm)
    gb, ga = ctx.pack_weights(dev(W))
    assert np.array_equal(bits_from_dev(gb), bitsT)
    np.testing.assert_allclose(ga.cpu().numpy(), alpha, rtol=1e-6)


@pytest.mark.parametrize("n,d,pad", [(1, 5, 0), (2, 47, 3), (5000, 77, 0), (4099, 256, 8), (700, 1433, 0), (300, 3703, 5),
                                     (40000, 1, 0), (2449029, 3, 1)])
def test_col_stats(ctx, n, d, pad):
    """Batch statistics of Sec. 4.4 against the oracle (two passes in double): any width, rows with a leading
    dimension larger than the width, a single row, a constant column (variance exactly 0, scale = eps^-1/2) and a
    column with an offset a thousand times its spread."""
    rng = np.random.default_rng(9 + n + d)
    H = (rng.standard_normal((n, d)) * 3 + 1.5).astype(np.float32)
    H[:, 0] = 3.25                                              # constant
    if d > 2:
        H[:, 2] = (1000.0 + rng.standard_normal(n)).astype(np.float32)
    shift, scale = oracle.col_stats(H)
    buf = np.full((n, d + pad), np.float32(7e9))                # whatever lies beyond a row's d columns is not read
    buf[:, :d] = H
    gs, gc = ctx.col_stats(dev(buf)[:, :d])
    np.testing.assert_allclose(gs.cpu().numpy(), shift, rtol=1e-6, atol=1e-7)
    np.testing.assert_allclose(gc.cpu().numpy(), scale, rtol=1e-6)
    assert gc[0].item() == pytest.approx(1e-5 ** -0.5, rel=1e-6)


# --------------------------------------------------------------------------- one layer, oracle-fed

LAYER_SHAPES = [(200, 1500, 1, 1), (300, 2500, 33, 7), (500, 6000, 100, 256), (400, 5000, 602, 256),
                (350, 3000, 1433, 64), (250, 2000, 3703, 64), (600, 9000, 256, 47), (600, 9000, 256, 41),
                (700, 5000, 64, 3), (450, 4000, 64, 6), (300, 3000, 256, 256), (260, 3000, 127, 100),
                (260, 3000, 128, 512), (300, 3000, 64, 200)]


@pytest.mark.parametrize("fmt", FORMATS)
@pytest.mark.parametrize("n,e,d_in,d_out", LAYER_SHAPES)
def test_layer_forward_against_oracle(ctx, B, fmt, n, e, d_in, d_out):
    check_layer_forward(ctx, B, fmt, n, e, d_in, d_out)


# half-dot bytes: every parity of d_in in range, both ends of the byte range, ragged column counts, several tiles
HALF_SHAPES = [(64, 300, 128, 129), (500, 6000, 129, 200), (700, 9000, 200, 256), (300, 4000, 255, 130),
               (300, 3000, 256, 256), (2000, 60000, 256, 200), (40000, 300000, 256, 256), (5000, 60000, 254, 256)]


@pytest.mark.parametrize("n,e,d_in,d_out", HALF_SHAPES)
def test_layer_forward_half_dot_bytes(ctx, B, n, e, d_in, d_out):
    check_layer_forward(ctx, B, 5, n, e, d_in, d_out)


# half-dot bytes in rows of 1, 2, 3, 4, 7 and 8 sixteen-byte vectors (the general stream): short and long rows,
# both parities of d_in, rows that end inside a group of positions
HALF_NARROW_SHAPES = [(64, 300, 128, 5), (500, 6000, 129, 16), (700, 9000, 200, 17), (300, 4000, 255, 32),
                      (3000, 30000, 256, 47), (2000, 120000, 256, 47), (40000, 300000, 256, 47), (900, 9000, 254, 64),
                      (1500, 40000, 256, 100), (5000, 60000, 256, 128), (600, 2400, 256, 41), (2000, 6000, 256, 100)]


@pytest.mark.parametrize("n,e,d_in,d_out", HALF_NARROW_SHAPES)
def test_layer_forward_half_dot_bytes_narrow_rows(ctx, B, n, e, d_in, d_out):
    check_layer_forward(ctx, B, 5, n, e, d_in, d_out)


def test_half_dot_bytes_at_the_ends_of_the_byte_range(ctx, B):
    """Rows equal to a weight column (dot = +256) and to its complement (dot = -256): the stored bytes reach
    +127 and -128; the reconstructed sums must still be exact."""
    n, d_in, d_out = 300, 256, 256
    rng = np.random.default_rng(12)
    _, _, g = small_graph(n, 3000, 12)
    W = rng.standard_normal((d_in, d_out)).astype(np.float32)
    H = rng.standard_normal((n, d_in)).astype(np.float32)
    H[0] = np.abs(H[0]) * np.where(W[:, 0] >= 0, 1, -1)        # same signs as column 0
    H[1] = -np.abs(H[1]) * np.where(W[:, 1] >= 0, 1, -1)       # opposite signs to column 1
    t = oracle.layer_forward(g, oracle.Layer(W), H)
    assert t.dot[0, 0] == 256 and t.dot[1, 1] == -256
    ctx.set_option(B.OPT_ZETA_FORMAT, 5)
    G = device_graph(B, g)
    layer = B.make_layer(d_in, d_out, bits_to_dev(t.bitsT), dev(t.alpha))
    out = ctx.layer_forward(G, layer, bits_to_dev(t.bits), dev(t.beta), want_h=True, debug=True)
    ctx.sync_check()
    assert np.array_equal(out["dot"].cpu().numpy(), t.dot)
    assert_close(out["h"], t.H_out, "H' (half-dot bytes, extreme dots)")


BYTE_ROW_SHAPES = [(3, 500, 6000, 100, 200), (3, 300, 3000, 127, 256), (3, 40000, 300000, 64, 130),
                   (5, 500, 6000, 129, 200), (5, 300, 3000, 256, 256), (5, 40000, 300000, 256, 256)]


# many rows of one or two entries (chunks limited by their eight row segments), a row count that is a multiple of
# the run length and one just above, ragged widths
BYTE_ROW_SHAPES_TC = [(3, 31 * 40, 700, 100, 256), (3, 31 * 40 + 1, 4000, 127, 129), (5, 5000, 5200, 256, 256),
                      (5, 2000, 150000, 200, 177), (5, 64, 2000, 256, 241), (3, 3, 4, 64, 256), (3, 3, 2, 100, 130)]


@pytest.mark.parametrize("path", [1, 2, 3])
@pytest.mark.parametrize("fmt,n,e,d_in,d_out", BYTE_ROW_SHAPES + BYTE_ROW_SHAPES_TC)
def test_byte_rows_as_integer_products(ctx, B, path, fmt, n, e, d_in, d_out):
    """The aggregations of 129..256 byte columns: the fp32 FMA stream (1) and the exact integer products with
    fixed-point edge weights on the tensor cores (2: mma.sync, operands in registers; 3: tcgen05, operands gathered
    straight into shared memory, digit sums in tensor memory)."""
    ctx.set_option(B.OPT_BYTE_AGGREGATION, path)
    try:
        check_layer_forward(ctx, B, fmt, n, e, d_in, d_out)
    finally:
        ctx.set_option(B.OPT_BYTE_AGGREGATION, 0)


@pytest.mark.parametrize("path", [2, 3])
@pytest.mark.parametrize("fmt,d_in", [(3, 100), (5, 256), (5, 201)])
@pytest.mark.parametrize("span", [0, 12, 40])
def test_byte_rows_signed_edge_values_of_wide_range(ctx, B, path, fmt, d_in, span):
    """Edge values of both signs spread over 2^-span .. 2^span inside every row: the fixed-point weights of the
    integer products take their scale from the largest weight of a piece of the row (path 2 opens a new segment as a
    larger weight arrives, path 3 scales every row segment of a chunk by its own maximum), and the sign rides in the
    digits.  The bound below is this test's own: the normalized adjacency never has such values, and the library's
    tolerance of 1e-4 + 1e-5 |x| is an absolute one that weights of 2^40 cannot meet in fp32 at all."""
    n, d_out = 600, 256
    rng = np.random.default_rng(5 + span)
    _, _, g = small_graph(n, 24000, 31)                      # about 80 entries per row: several windows
    g.val[:] = (g.val * np.exp2(rng.integers(-span, span + 1, g.val.shape)) * rng.choice([-1.0, 1.0], g.val.shape)).astype(np.float32)
    H = rng.standard_normal((n, d_in)).astype(np.float32)
    W = (rng.standard_normal((d_in, d_out)) * d_in ** -0.5).astype(np.float32)
    t = oracle.layer_forward(g, oracle.Layer(W), H)
    ctx.set_option(B.OPT_ZETA_FORMAT, fmt)
    ctx.set_option(B.OPT_BYTE_AGGREGATION, path)
    G = device_graph(B, g)
    layer = B.make_layer(d_in, d_out, bits_to_dev(t.bitsT), dev(t.alpha))
    try:
        out = ctx.layer_forward(G, layer, bits_to_dev(t.bits), dev(t.beta), want_h=True, debug=True)
        ctx.sync_check()
    finally:
        ctx.set_option(B.OPT_BYTE_AGGREGATION, 0)
    assert np.array_equal(out["dot"].cpu().numpy(), t.dot)
    ref = t.H_out
    got = out["h"].cpu().numpy().astype(np.float64)
    # fp32 summation is good to a few ulps of the sum of the terms' magnitudes; the fixed-point weights of the integer
    # products add at most 2^-28 of the row's largest weight per unit of |dot| (29 significant bits for the largest
    # weight of a segment's first window)
    A = np.zeros((n, n))
    for i in range(n):
        A[i, g.colidx[g.rowptr[i]:g.rowptr[i + 1]]] = np.abs(g.val[g.rowptr[i]:g.rowptr[i + 1]])
    Wabs = A * t.beta[None, :].astype(np.float64)
    adot = np.abs(t.dot).astype(np.float64)
    bound = (Wabs @ adot) * np.abs(t.alpha)[None, :]
    fixed = Wabs.max(axis=1)[:, None] * ((A > 0) @ adot) * np.abs(t.alpha)[None, :]
    assert np.all(np.abs(got - ref) <= 1e-5 * np.abs(ref) + 4e-6 * bound + 2.0 ** -27 * fixed + 1e-30)


# a network's last layer (fp32 output only) with 33..64 byte columns: the stream with one stored entry per lane
@pytest.mark.parametrize("d_in", [128, 256])
@pytest.mark.parametrize("d_out", [1, 4, 5, 8, 16])
def test_half_dot_bytes_asked_for_on_tiny_widths_stay_inside_an_exactly_sized_workspace(B, d_in, d_out):
    """Half-dot bytes keep two side arrays behind the byte rows inside the zeta scratch.  For d_out <= 4 they do not
    fit there (an fp32 row is no longer than a byte row), so the format falls back; from d_out = 5 they fit.  Either
    way the layer must match the oracle and must not write past a workspace of exactly bigcn_workspace_bytes()."""
    n = 300
    rng = np.random.default_rng(17 * d_in + d_out)
    _, _, g = small_graph(n, 2500, 77)
    H = rng.standard_normal((n, d_in)).astype(np.float32)
    W = (rng.standard_normal((d_in, d_out)) * d_in ** -0.5).astype(np.float32)
    t = oracle.layer_forward(g, oracle.Layer(W), H)
    ctx = B.BiGCN(0)
    ctx.set_option(B.OPT_ZETA_FORMAT, 5)
    need = ctx.workspace_bytes(n, g.nnz, [d_in, d_out])
    guard = 1 << 16
    buf = torch.full((need + guard,), 0xAB, dtype=torch.uint8, device="cuda")
    ctx.workspace = buf                                         # keeps the tensor alive; the library sees `need` bytes only
    ctx._check(ctx.lib.bigcn_set_workspace(ctx.h, ctypes.c_void_p(buf.data_ptr()), need))
    G = device_graph(B, g)
    layer = B.make_layer(d_in, d_out, bits_to_dev(t.bitsT), dev(t.alpha))
    for _ in range(2):                                          # the second call finds the first one's leftovers
        out = ctx.layer_forward(G, layer, bits_to_dev(t.bits), dev(t.beta), want_h=True, debug=True)
        ctx.sync_check()
        assert ctx.workspace is buf
        assert np.array_equal(out["dot"].cpu().numpy(), t.dot)
        assert_close(out["h"], t.H_out, "H'")
        assert bool((buf[need:] == 0xAB).all()), "bytes behind the workspace were written"
    ctx.close()


LAST_LAYER_SHAPES = [(5, 3000, 30000, 256, 47), (5, 2000, 120000, 256, 47), (5, 40000, 400000, 256, 41), (5, 900, 9000, 129, 33),
                     (5, 900, 9000, 254, 64), (5, 1500, 40000, 200, 48), (3, 3000, 30000, 100, 47), (3, 900, 20000, 127, 64),
                     (5, 64, 300, 256, 47), (5, 2000, 5000, 256, 47)]


@pytest.mark.parametrize("fmt,n,e,d_in,d_out", LAST_LAYER_SHAPES)
def test_last_layer_narrow_byte_rows(ctx, B, fmt, n, e, d_in, d_out):
    rng = np.random.default_rng(n + d_in + d_out)
    _, _, g = small_graph(n, e, 300 + n)
    H = rng.standard_normal((n, d_in)).astype(np.float32)
    W = (rng.standard_normal((d_in, d_out)) * d_in ** -0.5).astype(np.float32)
    t = oracle.layer_forward(g, oracle.Layer(W), H)
    ctx.set_option(B.OPT_ZETA_FORMAT, fmt)
    G = device_graph(B, g)
    layer = B.make_layer(d_in, d_out, bits_to_dev(t.bitsT), dev(t.alpha))
    out = ctx.layer_forward(G, layer, bits_to_dev(t.bits), dev(t.beta), want_h=True, debug=True)
    ctx.sync_check()
    assert np.array_equal(out["dot"].cpu().numpy(), t.dot)
    assert_close(out["h"], t.H_out, "H' (last layer, format %d)" % fmt)
    again = ctx.layer_forward(G, layer, bits_to_dev(t.bits), dev(t.beta), want_h=True)["h"]
    assert torch.equal(again, out["h"])                       # run-to-run deterministic


# hidden layers of 33..64 columns (re-binarized for a next layer) on graphs whose rows are not much shorter than a pass:
# byte rows and the one-entry-per-lane stream by default; 64-byte rows that carry the node factor where the
# tensor-core contraction runs (n * d_out >= 2^20); both byte formats; with and without the fp32 output
HIDDEN_NARROW_SHAPES = [(0, 900, 9000, 254, 64), (0, 3000, 30000, 100, 47), (0, 40000, 400000, 256, 47), (0, 40000, 400000, 100, 64),
                        (0, 40000, 400000, 127, 33), (0, 24000, 400000, 200, 60), (5, 1500, 40000, 256, 48), (3, 900, 20000, 127, 61),
                        (0, 2000, 5000, 256, 47)]


@pytest.mark.parametrize("fmt,n,e,d_in,d_out", HIDDEN_NARROW_SHAPES)
def test_hidden_layer_narrow_byte_rows(ctx, B, fmt, n, e, d_in, d_out):
    check_layer_forward(ctx, B, fmt, n, e, d_in, d_out)
    # the same layer without the fp32 output: bits and beta only
    rng = np.random.default_rng(n + 3 * d_in + 7 * d_out)
    _, _, g = small_graph(n, e, 100 + n)
    H = rng.standard_normal((n, d_in)).astype(np.float32)
    W = (rng.standard_normal((d_in, d_out)) * d_in ** -0.5).astype(np.float32)
    W2 = rng.standard_normal((d_out, 4)).astype(np.float32)
    t = oracle.layer_forward(g, oracle.Layer(W), H)
    nshift, nscale = oracle.col_stats(t.H_out)
    Fn, beta_n = oracle.binarize_rows(t.H_out, nshift, nscale)
    G = device_graph(B, g)
    layer = B.make_layer(d_in, d_out, bits_to_dev(t.bitsT), dev(t.alpha))
    nxt = B.make_layer(d_out, 4, bits_to_dev(oracle.pack_cols(oracle.binarize_cols(W2)[0])), dev(np.ones(4, np.float32)),
                       dev(nshift), dev(nscale))
    out = ctx.layer_forward(G, layer, bits_to_dev(t.bits), dev(t.beta), want_h=False, next_layer=nxt)
    ctx.sync_check()
    flips, bad, total = flip_report(bits_from_dev(out["next_bits"]), Fn, t.H_out, nshift)
    assert bad == 0 and flips <= max(2, total // 2000)
    nb = bits_from_dev(out["next_bits"])
    if d_out % 32:
        assert (nb[:, d_out // 32] >> (d_out % 32) == 0).all()
    assert (nb[:, (d_out + 31) // 32:] == 0).all()
    np.testing.assert_allclose(out["next_beta"].cpu().numpy(), beta_n, rtol=RTOL, atol=ATOL)


@pytest.mark.parametrize("fmt,d_in", [(5, 256), (3, 100)])
def test_hidden_layer_narrow_byte_rows_hub_row(ctx, B, fmt, d_in):
    """One row with n entries in a hidden layer of 47 columns: the block finishes the row and re-binarizes it."""
    n, d_out = 3000, 47
    rng = np.random.default_rng(79)
    rp, ci = synth.power_law_graph(n, 30000, 79)
    src, dst = synth.edge_list(rp, ci)
    src = np.concatenate([src, np.zeros(n - 1, np.int32)])
    dst = np.concatenate([dst, np.arange(1, n, dtype=np.int32)])
    g = oracle.normalize_adjacency(n, src, dst)
    H = rng.standard_normal((n, d_in)).astype(np.float32)
    W = (rng.standard_normal((d_in, d_out)) * 0.1).astype(np.float32)
    W2 = rng.standard_normal((d_out, 4)).astype(np.float32)
    t = oracle.layer_forward(g, oracle.Layer(W), H)
    nshift, nscale = oracle.col_stats(t.H_out)
    Fn, beta_n = oracle.binarize_rows(t.H_out, nshift, nscale)
    ctx.set_option(B.OPT_ZETA_FORMAT, fmt)
    G = device_graph(B, g)
    layer = B.make_layer(d_in, d_out, bits_to_dev(t.bitsT), dev(t.alpha))
    nxt = B.make_layer(d_out, 4, bits_to_dev(oracle.pack_cols(oracle.binarize_cols(W2)[0])), dev(np.ones(4, np.float32)),
                       dev(nshift), dev(nscale))
    try:
        for thr in (0, 8, 100000):
            ctx.set_option(B.OPT_LONG_ROW, thr)
            out = ctx.layer_forward(G, layer, bits_to_dev(t.bits), dev(t.beta), want_h=True, next_layer=nxt)
            ctx.sync_check()
            assert_close(out["h"], t.H_out, "H' (threshold %d)" % thr)
            flips, bad, total = flip_report(bits_from_dev(out["next_bits"]), Fn, t.H_out, nshift)
            assert bad == 0 and flips <= max(2, total // 2000)
            nb = bits_from_dev(out["next_bits"])
            assert (nb[:, 1] >> 15 == 0).all() and (nb[:, 2:] == 0).all()
            np.testing.assert_allclose(out["next_beta"].cpu().numpy(), beta_n, rtol=RTOL, atol=ATOL)
    finally:
        ctx.set_option(B.OPT_LONG_ROW, 0)


@pytest.mark.parametrize("d_out", [256, 47])
def test_half_dot_bytes_hub_row_split_across_the_block(ctx, B, d_out):
    """One row with n entries under half-dot bytes: slices of a long row hand back reconstructed partial sums."""
    n, d_in = 3000, 256
    rng = np.random.default_rng(78)
    rp, ci = synth.power_law_graph(n, 30000, 78)
    src, dst = synth.edge_list(rp, ci)
    src = np.concatenate([src, np.zeros(n - 1, np.int32)])
    dst = np.concatenate([dst, np.arange(1, n, dtype=np.int32)])
    g = oracle.normalize_adjacency(n, src, dst)
    H = rng.standard_normal((n, d_in)).astype(np.float32)
    W = (rng.standard_normal((d_in, d_out)) * 0.1).astype(np.float32)
    t = oracle.layer_forward(g, oracle.Layer(W), H)
    ctx.set_option(B.OPT_ZETA_FORMAT, 5)
    G = device_graph(B, g)
    layer = B.make_layer(d_in, d_out, bits_to_dev(t.bitsT), dev(t.alpha))
    for path in (1, 2, 3):
        ctx.set_option(B.OPT_BYTE_AGGREGATION, path)
        try:
            for thr in (0, 8, 100000):
                ctx.set_option(B.OPT_LONG_ROW, thr)
                out = ctx.layer_forward(G, layer, bits_to_dev(t.bits), dev(t.beta), want_h=True)
                assert_close(out["h"], t.H_out, "H' (path %d, threshold %d)" % (path, thr))
        finally:
            ctx.set_option(B.OPT_BYTE_AGGREGATION, 0)
            ctx.set_option(B.OPT_LONG_ROW, 0)


# shapes the tensor-core contraction covers (d_in, d_out <= 256): tile tails, one row, several tiles per CTA
TC_SHAPES = [(5, 6, 256, 256), (127, 900, 256, 256), (128, 900, 100, 256), (129, 900, 256, 47), (1000, 9000, 200, 130),
             (40000, 200000, 256, 256), (39000, 150000, 100, 64)]


@pytest.mark.parametrize("fmt", [1, 2, 3, 4])
@pytest.mark.parametrize("n,e,d_in,d_out", TC_SHAPES + [s for s in LAYER_SHAPES if s[2] <= 256 and s[3] <= 256])
def test_layer_forward_tensor_core_contraction(ctx, B, fmt, n, e, d_in, d_out):
    ctx.set_option(B.OPT_CONTRACTION, 2)          # also below the size from which it is the default
    try:
        check_layer_forward(ctx, B, fmt, n, e, d_in, d_out)
    finally:
        ctx.set_option(B.OPT_CONTRACTION, 0)


@pytest.mark.parametrize("fmt", [1, 3, 4])
@pytest.mark.parametrize("n,e,d_in,d_out", [s for s in LAYER_SHAPES if s[2] <= 256 and s[3] <= 256])
def test_layer_forward_on_the_bit_count_pipe(ctx, B, fmt, n, e, d_in, d_out):
    """The library's other contraction path (XOR + bit count on the integer pipe) for the shapes that take the
    tensor cores by default."""
    ctx.set_option(B.OPT_CONTRACTION, 1)
    try:
        check_layer_forward(ctx, B, fmt, n, e, d_in, d_out)
    finally:
        ctx.set_option(B.OPT_CONTRACTION, 0)


def check_layer_forward(ctx, B, fmt, n, e, d_in, d_out):
    rng = np.random.default_rng(n + 3 * d_in + 7 * d_out)
    _, _, g = small_graph(n, e, 100 + n)
    H = rng.standard_normal((n, d_in)).astype(np.float32)
    W = (rng.standard_normal((d_in, d_out)) * d_in ** -0.5).astype(np.float32)
    W2 = rng.standard_normal((d_out, 4)).astype(np.float32)
    t = oracle.layer_forward(g, oracle.Layer(W), H)
    nshift, nscale = oracle.col_stats(t.H_out)
    Fn, beta_n = oracle.binarize_rows(t.H_out, nshift, nscale)

    ctx.set_option(B.OPT_ZETA_FORMAT, fmt)
    G = device_graph(B, g)
    layer = B.make_layer(d_in, d_out, bits_to_dev(t.bitsT), dev(t.alpha))
    nxt = B.make_layer(d_out, 4, bits_to_dev(oracle.pack_cols(oracle.binarize_cols(W2)[0])), dev(np.ones(4, np.float32)),
                       dev(nshift), dev(nscale))
    out = ctx.layer_forward(G, layer, bits_to_dev(t.bits), dev(t.beta), want_h=True, next_layer=nxt, debug=True)
    ctx.sync_check()
    assert np.array_equal(out["dot"].cpu().numpy(), t.dot)                 # integers: exact
    assert np.array_equal(out["zeta"].cpu().numpy(), t.zeta)               # same two fp32 products: exact
    assert_close(out["h"], t.H_out, "H'")
    flips, bad, total = flip_report(bits_from_dev(out["next_bits"]), Fn, t.H_out, nshift)
    assert bad == 0, "%d sign flips away from the threshold (of %d flips, %d bits)" % (bad, flips, total)
    assert flips <= max(2, total // 2000)
    # pad bits of the re-binarized rows are zero
    nb = bits_from_dev(out["next_bits"])
    if d_out % 32:
        assert (nb[:, d_out // 32] >> (d_out % 32) == 0).all()
    assert (nb[:, (d_out + 31) // 32:] == 0).all()
    np.testing.assert_allclose(out["next_beta"].cpu().numpy(), beta_n, rtol=RTOL, atol=ATOL)
    # the same layer with only the sign bits and beta wanted (how a hidden layer runs inside bigcn_forward; for byte
    # rows of 129..256 columns that launch takes the tcgen05 aggregation by default)
    outb = ctx.layer_forward(G, layer, bits_to_dev(t.bits), dev(t.beta), want_h=False, next_layer=nxt)
    ctx.sync_check()
    nb = bits_from_dev(outb["next_bits"])
    flips, bad, total = flip_report(nb, Fn, t.H_out, nshift)
    assert bad == 0, "bits only: %d sign flips away from the threshold (of %d flips, %d bits)" % (bad, flips, total)
    assert flips <= max(2, total // 2000)
    if d_out % 32:
        assert (nb[:, d_out // 32] >> (d_out % 32) == 0).all()
    assert (nb[:, (d_out + 31) // 32:] == 0).all()
    np.testing.assert_allclose(outb["next_beta"].cpu().numpy(), beta_n, rtol=RTOL, atol=ATOL)


@pytest.mark.parametrize("fmt", FORMATS)
def test_layer_forward_hub_rows_split_across_the_block(ctx, B, fmt):
    """A star plus a random graph: one row holds n entries.  With a tiny long-row threshold every
    moderately long row takes the block-cooperative path; results must not change."""
    n, d_in, d_out = 3000, 100, 256
    rng = np.random.default_rng(77)
    rp, ci = synth.power_law_graph(n, 30000, 77)
    src, dst = synth.edge_list(rp, ci)
    src = np.concatenate([src, np.zeros(n - 1, np.int32)])
    dst = np.concatenate([dst, np.arange(1, n, dtype=np.int32)])
    g = oracle.normalize_adjacency(n, src, dst)
    assert (np.diff(g.rowptr)).max() == n
    H = rng.standard_normal((n, d_in)).astype(np.float32)
    W = (rng.standard_normal((d_in, d_out)) * 0.1).astype(np.float32)
    t = oracle.layer_forward(g, oracle.Layer(W), H)
    ctx.set_option(B.OPT_ZETA_FORMAT, fmt)
    G = device_graph(B, g)
    layer = B.make_layer(d_in, d_out, bits_to_dev(t.bitsT), dev(t.alpha))
    outs = []
    for thr in (0, 8, 100000):       # default threshold, nearly every row long, no row long
        ctx.set_option(B.OPT_LONG_ROW, thr)
        out = ctx.layer_forward(G, layer, bits_to_dev(t.bits), dev(t.beta), want_h=True)
        assert_close(out["h"], t.H_out, "H' (threshold %d)" % thr)
        outs.append(out["h"].clone())
    again = ctx.layer_forward(G, layer, bits_to_dev(t.bits), dev(t.beta), want_h=True)["h"]
    assert torch.equal(again, outs[-1])          # run-to-run deterministic


def test_layer_on_pm1_inputs_is_the_gcn_layer(ctx, B):
    """H, W in {+-1}: the scalars are 1 and the layer is exactly A_tilde (H W) (Eq. 1, no activation)."""
    rng = np.random.default_rng(21)
    n, d, c = 300, 45, 5
    _, _, g = small_graph(n, 2000, 21)
    H = rng.choice(np.array([-1.0, 1.0], np.float32), size=(n, d))
    W = rng.choice(np.array([-1.0, 1.0], np.float32), size=(d, c))
    G = device_graph(B, g)
    bits, beta = ctx.pack_features(dev(H))
    bitsT, alpha = ctx.pack_weights(dev(W))
    assert (beta == 1).all() and (alpha == 1).all()
    out = ctx.layer_forward(G, B.make_layer(d, c, bitsT, alpha), bits, beta)
    A = torch.sparse_csr_tensor(dev(g.rowptr), dev(g.colidx).long(), dev(g.val).double(), size=(n, n))
    ref = (A.to_dense() @ (dev(H).double() @ dev(W).double()))
    assert_close(out["h"], ref.float().cpu(), "GCN special case")


def test_isolated_nodes_and_empty_graph(ctx, B):
    n, d_in, d_out = 37, 50, 9
    rng = np.random.default_rng(3)
    e = np.zeros(0, np.int32)
    g = oracle.normalize_adjacency(n, e, e)                        # A_tilde = I  =>  H' = zeta
    H = rng.standard_normal((n, d_in)).astype(np.float32)
    W = rng.standard_normal((d_in, d_out)).astype(np.float32)
    t = oracle.layer_forward(g, oracle.Layer(W), H)
    G = device_graph(B, g)
    out = ctx.layer_forward(G, B.make_layer(d_in, d_out, bits_to_dev(t.bitsT), dev(t.alpha)), bits_to_dev(t.bits),
                            dev(t.beta), debug=True)
    assert_close(out["h"], t.H_out, "identity adjacency")
    assert_close(out["h"], out["zeta"].cpu(), "H' = zeta")
    # n = 0 is a no-op
    G0 = B.make_graph(torch.zeros(1, dtype=torch.int64).cuda(), torch.zeros(0, dtype=torch.int32).cuda(),
                      torch.zeros(0).cuda())
    lay = B.make_layer(d_in, d_out, bits_to_dev(t.bitsT), dev(t.alpha))
    logits = ctx.forward(G0, [lay], torch.zeros((0, d_in)).cuda())
    assert logits.shape == (0, d_out)


def test_gather_only_probe(ctx, B):
    """The measurement aid that reads every stored entry's operand row and nothing else: runs, times, validates."""
    _, _, g = small_graph(5000, 60000, 11)
    G = device_graph(B, g)
    for rb in (16, 64, 256, 512):
        assert ctx.measure_gather_peak(G, rb) > 0.0
    for bad in (0, 8, 48, 1024):
        with pytest.raises(B.BigcnError):
            ctx.measure_gather_peak(G, bad)
    ctx.sync_check()


def test_argument_errors_are_reported_not_launched(ctx, B):
    import ctypes
    n, d_in, d_out = 10, 40, 5
    _, _, g = small_graph(n, 30, 1)
    G = device_graph(B, g)
    bitsT = torch.zeros((d_out, 4), dtype=torch.int32).cuda()
    alpha = torch.ones(d_out).cuda()
    lay = B.make_layer(d_in, d_out, bitsT, alpha)
    before = ctx.launch_count()
    with pytest.raises(B.BigcnError) as e:                      # no workspace large enough: shrink it
        ctx.lib.bigcn_set_workspace(ctx.h, None, 0)
        ctx._check(ctx.lib.bigcn_forward(ctx.h, ctypes.byref(G.c), B._layer_array([lay]), 1,
                                         ctypes.c_void_p(alpha.data_ptr()), d_in, ctypes.c_void_p(alpha.data_ptr()), d_out, None))
    assert e.value.status == 5
    ctx.workspace = None
    bad = B.make_layer(d_in, 0, bitsT, alpha)
    with pytest.raises(B.BigcnError) as e:
        ctx.forward(G, [bad], torch.zeros((n, d_in)).cuda())
    assert e.value.status == 2
    two = [lay, B.make_layer(d_out + 1, 3, bitsT, alpha)]          # widths do not chain
    with pytest.raises(B.BigcnError) as e:
        ctx.forward(G, two, torch.zeros((n, d_in)).cuda())
    assert e.value.status == 2
    with pytest.raises(B.BigcnError) as e:                      # misaligned packed input
        ctx._check(ctx.lib.bigcn_pack_features(ctx.h, ctypes.c_void_p(alpha.data_ptr()), 1, 4, 4, None, None,
                                               ctypes.c_void_p(bitsT.data_ptr() + 4), 4, ctypes.c_void_p(alpha.data_ptr())))
    assert e.value.status == 3
    assert ctx.launch_count() == before


# --------------------------------------------------------------------------- whole networks

NETS = [("c1", None), ("c2", None), ("c3", None), ("c4", 0.01), ("c5", 0.004)]


@pytest.fixture(scope="module", params=NETS, ids=lambda p: p[0] if p[1] is None else "%s@%g" % p)
def net(request):
    name, scale = request.param
    wl = synth.make_workload(name, scale=scale, device="cuda")
    return oracle_run(wl)


@pytest.mark.parametrize("fmt", FORMATS)
def test_network_layer_by_layer_oracle_fed(B, net, fmt):
    """Each layer is fed the oracle's own input (packed bits and beta); bits and dots exact, fp32
    within tolerance, re-binarized bits equal up to threshold-adjacent flips."""
    ctx = B.BiGCN(0)
    ctx.set_option(B.OPT_ZETA_FORMAT, fmt)
    G = device_graph(B, net.graph)
    layers = device_layers_from_oracle(B, net)
    L = len(layers)
    for l in range(L):
        t = net.traces[l]
        nxt = layers[l + 1] if l + 1 < L else None
        out = ctx.layer_forward(G, layers[l], bits_to_dev(t.bits), dev(t.beta), want_h=True, next_layer=nxt, debug=True)
        assert torch.equal(out["dot"].cpu(), torch.from_numpy(t.dot))
        assert torch.equal(out["zeta"].cpu(), torch.from_numpy(t.zeta))
        assert_close(out["h"], t.H_out, "layer %d output" % l)
        if nxt is not None:
            tn = net.traces[l + 1]
            flips, bad, total = flip_report(bits_from_dev(out["next_bits"]), tn.F, t.H_out, net.layers[l + 1].in_shift)
            assert bad == 0 and flips <= max(2, total // 2000), (flips, bad, total)
            np.testing.assert_allclose(out["next_beta"].cpu().numpy(), tn.beta, rtol=RTOL, atol=ATOL)
    ctx.sync_check()
    ctx.close()


@pytest.mark.parametrize("fmt", FORMATS)
def test_network_end_to_end(B, net, fmt):
    """From fp32 features and fp32 weights through the library's own packers to logits."""
    wl = net.wl
    ctx = B.BiGCN(0)
    ctx.set_option(B.OPT_ZETA_FORMAT, fmt)
    G = ctx.normalize_adjacency(wl.rowptr.cuda(), wl.colidx.cuda())
    shifts = [dev(l.in_shift) if l.in_shift is not None else None for l in net.layers]
    scales = [dev(l.in_scale) if l.in_scale is not None else None for l in net.layers]
    layers = ctx.prepare_layers([w.cuda() for w in wl.W], shifts, scales)
    X = wl.X.cuda()
    # first-layer bits must be exact (sign(x - mu) is decided in the same fp32 arithmetic)
    xb, xbeta = ctx.pack_features(X, shifts[0], scales[0])
    assert np.array_equal(bits_from_dev(xb), net.traces[0].bits)
    logits, st = ctx.forward(G, layers, X, stats=True)
    ref = torch.from_numpy(net.logits)
    err = (logits.cpu().double() - ref.double()).abs()
    allow = ATOL + RTOL * ref.double().abs()
    frac_out = (err > allow).double().mean().item()
    agree = (logits.cpu().argmax(1) == ref.argmax(1)).double().mean().item()
    print("\n[%s fmt %d] max|err| %.3g, share outside tolerance %.3g, argmax agreement %.6f, launches %d, %.3f ms"
          % (wl.spec.name, fmt, err.max().item(), frac_out, agree, st.launches, st.ms_total))
    # a sign flip at a re-binarization moves the logits downstream of it beyond the per-element
    # tolerance: every logit row that no flip reaches must be within tolerance, every flip must sit at
    # the threshold, and the predictions must agree
    rep = end_to_end_with_flip_accounting(ctx, G, layers, net, X)
    print("[%s fmt %d] %s" % (wl.spec.name, fmt, rep))
    assert agree >= 0.995 and abs(rep["logits_outside_tolerance"] - frac_out) < 1e-12
    assert st.launches == 1 + 2 * len(layers)
    # same result from pre-packed input and from host buffers
    l2 = ctx.forward_packed(G, layers, xb, xbeta)
    assert torch.equal(l2, logits)
    xh = wl.X.cpu().pin_memory()
    oh = torch.empty((wl.n, wl.spec.dims[-1]), dtype=torch.float32).pin_memory()
    ctx.forward_host(G, layers, xh, oh)
    assert torch.equal(oh, logits.cpu())
    # deterministic from run to run
    assert torch.equal(ctx.forward(G, layers, X), logits)
    ctx.sync_check()
    ctx.close()


def test_network_flip_rate_report(B, net):
    """End to end with the GPU's own intermediate results: how many re-binarized bits differ from the
    oracle's (reported; they can only sit next to the threshold)."""
    wl = net.wl
    ctx = B.BiGCN(0)
    G = device_graph(B, net.graph)
    layers = device_layers_from_oracle(B, net)
    bits, beta = bits_to_dev(net.traces[0].bits), dev(net.traces[0].beta)
    for l in range(len(layers) - 1):
        out = ctx.layer_forward(G, layers[l], bits, beta, want_h=False, next_layer=layers[l + 1])
        bits, beta = out["next_bits"], out["next_beta"]
        got = oracle.unpack_rows(bits_from_dev(bits), layers[l].d_out)
        flips = int((got != net.traces[l + 1].F).sum())
        print("\n[%s] layer %d -> %d: %d of %d bits flipped (%.3g)" % (wl.spec.name, l, l + 1, flips, got.size, flips / got.size))
        assert flips <= max(4, got.size // 1000)
    ctx.close()

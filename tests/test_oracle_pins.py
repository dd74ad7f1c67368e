"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU needed).

Each test checks the oracle against something other than itself: a brute-force search, a dense
numpy/scipy routine on a special case that reduces to it, a hand-worked graph, or a value the
paper prints.
"""
import itertools
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def dense_norm_adj(n, pairs):
    """D_hat^-1/2 (A + I) D_hat^-1/2 in float64, dense (Eq. 1, Sec. 3.1)."""
    A = np.zeros((n, n))
    for u, v in pairs:
        if u != v:
            A[u, v] = 1.0
            A[v, u] = 1.0
    A_hat = A + np.eye(n)
    d = A_hat.sum(1)
    return A_hat / np.sqrt(np.outer(d, d)), d


def to_dense(g):
    M = np.zeros((g.n, g.n))
    for i in range(g.n):
        for p in range(g.rowptr[i], g.rowptr[i + 1]):
            M[i, g.colidx[p]] += g.val[p]
    return M


def random_pairs(rng, n, m):
    return rng.integers(0, n, size=(m, 2)).astype(np.int32)


# ------------------------------------------------------------------ Sec. 4.1: optimal binarization

@pytest.mark.parametrize("t", [1, 2, 5, 9, 12])
def test_vector_binarization_is_the_brute_force_optimum(t):
    """argmin over all 2^t sign vectors and a fine alpha grid of ||V - alpha V_B||^2 is
    (sign(V), ||V||_1 / t): the closed form of Sec. 4.1."""
    rng = np.random.default_rng(100 + t)
    V = rng.standard_normal(t).astype(np.float32)
    F, beta = oracle.binarize_rows(V[None, :])
    B, alpha = oracle.binarize_cols(V[:, None])
    assert np.array_equal(F[0], B[:, 0])
    assert beta[0] == alpha[0]
    grid = np.linspace(0.0, float(np.abs(V).max()) * 1.5, 3001)
    best = (np.inf, None, None)
    for signs in itertools.product((-1.0, 1.0), repeat=t):
        s = np.asarray(signs)
        J = ((V[None, :].astype(np.float64) - grid[:, None] * s[None, :]) ** 2).sum(1)
        k = int(J.argmin())
        if J[k] < best[0]:
            best = (J[k], s, grid[k])
    assert np.array_equal(best[1].astype(np.int8), F[0])
    assert abs(best[2] - float(beta[0])) <= (grid[1] - grid[0])
    # and the oracle's (sign, scalar) is no worse than the best grid point
    J_or = ((V.astype(np.float64) - float(beta[0]) * F[0]) ** 2).sum()
    assert J_or <= best[0] + 1e-12


def test_scalars_are_l1_over_bucket_length_not_over_the_other_dimension():
    """beta_i = ||H_i,:||_1 / d_in and alpha_j = ||W_:,j||_1 / d_in (generic rule of Sec. 4.1);
    a rectangular case tells d_in from N and from d_out."""
    rng = np.random.default_rng(7)
    H = rng.standard_normal((5, 11)).astype(np.float32)
    W = rng.standard_normal((11, 3)).astype(np.float32)
    _, beta = oracle.binarize_rows(H)
    _, alpha = oracle.binarize_cols(W)
    np.testing.assert_allclose(beta, np.abs(H.astype(np.float64)).sum(1) / 11, rtol=1e-7)
    np.testing.assert_allclose(alpha, np.abs(W.astype(np.float64)).sum(0) / 11, rtol=1e-7)


def test_sign_convention_and_special_values():
    tiny = np.float32(1e-45)  # smallest denormal
    H = np.array([[0.0, -0.0, tiny, -tiny, 1.0, -1.0, np.inf, -np.inf]], np.float32)
    F, beta = oracle.binarize_rows(H[:, :6])
    assert F.tolist() == [[1, 1, 1, -1, 1, -1]]
    F2, _ = oracle.binarize_rows(H)
    assert F2.tolist() == [[1, 1, 1, -1, 1, -1, 1, -1]]
    B, _ = oracle.binarize_cols(H[:, :6].T.copy())
    assert B[:, 0].tolist() == [1, 1, 1, -1, 1, -1]
    Fn, _ = oracle.binarize_rows(np.array([[np.nan, 1.0]], np.float32))
    assert Fn.tolist() == [[-1, 1]]
    # an all-zero row: beta = 0, so its zeta row is 0 whatever the signs
    Z, bz = oracle.binarize_rows(np.zeros((1, 7), np.float32))
    assert bz[0] == 0.0 and (Z == 1).all()


# ------------------------------------------------------------------ Sec. 4.2.3: XNOR / bit count

@pytest.mark.parametrize("n,d_in,d_out", [(3, 1, 2), (4, 7, 3), (5, 31, 4), (6, 32, 5), (7, 33, 6),
                                           (9, 64, 7), (5, 100, 41), (4, 257, 3), (3, 1433, 7)])
def test_popcount_dot_equals_float_pm1_matmul(n, d_in, d_out):
    rng = np.random.default_rng(d_in * 131 + d_out)
    F = rng.choice(np.array([-1, 1], np.int8), size=(n, d_in))
    B = rng.choice(np.array([-1, 1], np.int8), size=(d_in, d_out))
    ref = (F.astype(np.float64) @ B.astype(np.float64)).astype(np.int64)   # library matmul of +-1 floats
    bits = oracle.pack_rows(F)
    bitsT = oracle.pack_cols(B)
    got_popc = oracle.dot_popc(bits, bitsT, d_in)
    got_pm1 = oracle.dot_pm1(F, B)
    assert np.array_equal(got_pm1, ref)
    assert np.array_equal(got_popc, ref)
    # dot = K - 2 * Hamming distance, computed here from the +-1 matrices directly
    ham = (F[:, :, None] != B[None, :, :]).sum(1)
    assert np.array_equal(got_popc, d_in - 2 * ham)
    assert ((got_popc - d_in) % 2 == 0).all() and (np.abs(got_popc) <= d_in).all()


def test_popcount_dot_extremes():
    d = 70
    F = np.ones((2, d), np.int8)
    F[1] = -1
    B = np.ones((d, 2), np.int8)
    B[:, 1] = -1
    got = oracle.dot_popc(oracle.pack_rows(F), oracle.pack_cols(B), d)
    assert got.tolist() == [[d, -d], [-d, d]]


@pytest.mark.parametrize("d", [1, 31, 32, 33, 100, 129])
def test_packing_layout_roundtrip_and_padding(d):
    rng = np.random.default_rng(d)
    F = rng.choice(np.array([-1, 1], np.int8), size=(6, d))
    bits = oracle.pack_rows(F)
    stride = bits.shape[1]
    assert stride % 4 == 0 and stride >= (d + 31) // 32 and stride == oracle.stride_words(d)
    assert np.array_equal(oracle.unpack_rows(bits, d), F)
    # layout: element 32 w + k is bit k of word w, +1 <-> 1, stated independently with numpy
    padded = np.zeros((6, stride * 32), np.uint8)
    padded[:, :d] = (F > 0)
    expect = np.packbits(padded.reshape(6, stride, 32), axis=2, bitorder="little")
    expect = expect.reshape(6, stride, 4).astype(np.uint32)
    expect = expect[..., 0] | (expect[..., 1] << 8) | (expect[..., 2] << 16) | (expect[..., 3] << 24)
    assert np.array_equal(bits, expect)
    # a 64-bit view is two consecutive words, low word first
    v64 = bits.view(np.uint64)
    assert np.array_equal(v64, bits[:, 0::2].astype(np.uint64) | (bits[:, 1::2].astype(np.uint64) << 32))
    # weights are packed transposed: row j of bitsT is column j of B
    B = F.T.copy()
    assert np.array_equal(oracle.pack_cols(B), bits)


def test_rescale_is_beta_times_alpha_times_dot():
    rng = np.random.default_rng(3)
    dot = rng.integers(-50, 50, size=(4, 6)).astype(np.int32)
    beta = rng.random(4).astype(np.float32)
    alpha = rng.random(6).astype(np.float32)
    z = oracle.rescale(dot, beta, alpha)
    expect = (beta[:, None] * alpha[None, :]).astype(np.float32) * dot.astype(np.float32)
    assert np.array_equal(z, expect.astype(np.float32))


# ------------------------------------------------------------------ Sec. 3: normalised adjacency

def _load_hand_graphs():
    graphs, cur = {}, None
    for line in open(os.path.join(GOLDEN, "path3_star4_adjacency.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        tok = line.split()
        if tok[0] == "graph":
            cur = {"n": int(tok[2]), "entries": []}
            graphs[tok[1]] = cur
        else:
            cur["entries"].append(tuple(int(t) for t in tok))
    return graphs


@pytest.mark.parametrize("name,pairs", [("path3", [(0, 1), (1, 2)]), ("star4", [(0, 1), (0, 2), (3, 0)])])
def test_hand_worked_adjacency(name, pairs):
    spec = _load_hand_graphs()[name]
    p = np.asarray(pairs, np.int32)
    g = oracle.normalize_adjacency(spec["n"], p[:, 0], p[:, 1])
    assert g.nnz == len(spec["entries"])
    M = to_dense(g)
    seen = np.zeros_like(M, dtype=bool)
    for i, j, di, dj in spec["entries"]:
        assert abs(M[i, j] - 1.0 / np.sqrt(di * dj)) < 1e-7
        seen[i, j] = True
    assert (M[~seen] == 0).all()


def test_adjacency_matches_dense_definition_with_messy_input():
    """Duplicates, both directions, one direction only and self pairs in the input all lead to
    the same undirected simple graph plus one self-loop per node."""
    rng = np.random.default_rng(11)
    n = 40
    pairs = random_pairs(rng, n, 150)
    pairs = np.concatenate([pairs, pairs[:30], pairs[:20, ::-1], np.stack([np.arange(5)] * 2, 1).astype(np.int32)])
    g = oracle.normalize_adjacency(n, pairs[:, 0], pairs[:, 1])
    dense, d_hat = dense_norm_adj(n, pairs.tolist())
    M = to_dense(g)
    np.testing.assert_allclose(M, dense, rtol=0, atol=2e-7)
    # CSR structure: ascending columns, no repeats, diagonal present
    for i in range(n):
        cols = g.colidx[g.rowptr[i]:g.rowptr[i + 1]]
        assert (np.diff(cols) > 0).all() and i in cols
    # invariants: symmetry, diag = 1/d_hat, A_tilde d_hat^1/2 = d_hat^1/2
    assert np.array_equal(M, M.T)
    np.testing.assert_allclose(np.diag(M), 1.0 / d_hat, rtol=1e-6)
    np.testing.assert_allclose(M @ np.sqrt(d_hat), np.sqrt(d_hat), rtol=1e-6)
    np.testing.assert_allclose(g.dinv, d_hat ** -0.5, rtol=1e-7)


def test_adjacency_degenerate_graphs():
    e = np.zeros(0, np.int32)
    g = oracle.normalize_adjacency(5, e, e)                 # no edges: A_tilde = I
    assert np.array_equal(to_dense(g), np.eye(5))
    n = 6                                                    # complete graph: every entry 1/n
    pairs = np.asarray(list(itertools.combinations(range(n), 2)), np.int32)
    g = oracle.normalize_adjacency(n, pairs[:, 0], pairs[:, 1])
    np.testing.assert_allclose(to_dense(g), np.full((n, n), 1.0 / n), rtol=1e-6)
    ring = np.asarray([(i, (i + 1) % 7) for i in range(7)], np.int32)   # regular: row sums are 1
    g = oracle.normalize_adjacency(7, ring[:, 0], ring[:, 1])
    np.testing.assert_allclose(to_dense(g).sum(1), np.ones(7), rtol=1e-6)
    with pytest.raises(ValueError):
        oracle.normalize_adjacency(3, np.asarray([0], np.int32), np.asarray([3], np.int32))


# ------------------------------------------------------------------ Sec. 4.2.3: aggregation

def test_spmm_equals_dense_product():
    rng = np.random.default_rng(5)
    n, d = 50, 9
    pairs = random_pairs(rng, n, 200)
    g = oracle.normalize_adjacency(n, pairs[:, 0], pairs[:, 1])
    zeta = rng.standard_normal((n, d)).astype(np.float32)
    dense = to_dense(g) @ zeta.astype(np.float64)
    got = oracle.spmm(g, zeta)
    np.testing.assert_allclose(got, dense, rtol=1e-6, atol=1e-7)
    part = oracle.spmm(g, zeta, 7, 23)
    assert np.array_equal(part, got[7:23])


def test_spmm_star_graph_by_hand():
    p = np.asarray([(0, 1), (0, 2), (0, 3)], np.int32)
    g = oracle.normalize_adjacency(4, p[:, 0], p[:, 1])
    z = np.asarray([[8.0], [2.0], [4.0], [6.0]], np.float32)
    # centre: 8/4 + (2+4+6)/sqrt(8); leaf k: z_k/2 + 8/sqrt(8)
    expect = np.asarray([[2.0 + 12.0 / np.sqrt(8.0)], [1.0 + 8 / np.sqrt(8.0)],
                         [2.0 + 8 / np.sqrt(8.0)], [3.0 + 8 / np.sqrt(8.0)]])
    np.testing.assert_allclose(oracle.spmm(g, z), expect, rtol=1e-6)


# ------------------------------------------------------------------ the whole layer

def test_layer_on_pm1_inputs_is_the_fp32_gcn_layer():
    """With H in {+-1}^(N x d) and W in {+-1}^(d x c) the scalars are 1 and the binarized layer is
    exactly the GCN layer A_tilde (H W) of Eq. 1 without activation."""
    rng = np.random.default_rng(21)
    n, d, c = 30, 45, 5
    pairs = random_pairs(rng, n, 90)
    g = oracle.normalize_adjacency(n, pairs[:, 0], pairs[:, 1])
    H = rng.choice(np.array([-1.0, 1.0], np.float32), size=(n, d))
    W = rng.choice(np.array([-1.0, 1.0], np.float32), size=(d, c))
    t = oracle.layer_forward(g, oracle.Layer(W), H)
    assert (t.beta == 1).all() and (t.alpha == 1).all()
    dense, _ = dense_norm_adj(n, pairs.tolist())
    np.testing.assert_allclose(t.H_out, dense @ (H.astype(np.float64) @ W), rtol=1e-6, atol=1e-6)
    t2 = oracle.layer_forward(g, oracle.Layer(W), H, use_pm1=True)
    assert np.array_equal(t.H_out, t2.H_out)


def test_layer_on_scaled_sign_matrices_is_exact_matmul():
    """H = diag(b) S and W = S' diag(a) with sign matrices S, S' and positive b, a: the binarized
    approximation is exact, so the layer equals A_tilde H W."""
    rng = np.random.default_rng(22)
    n, d, c = 25, 70, 4
    pairs = random_pairs(rng, n, 60)
    g = oracle.normalize_adjacency(n, pairs[:, 0], pairs[:, 1])
    b = (rng.random(n) + 0.5).astype(np.float32)
    a = (rng.random(c) + 0.5).astype(np.float32)
    S = rng.choice(np.array([-1.0, 1.0], np.float32), size=(n, d))
    S2 = rng.choice(np.array([-1.0, 1.0], np.float32), size=(d, c))
    H = b[:, None] * S
    W = S2 * a[None, :]
    t = oracle.layer_forward(g, oracle.Layer(W), H)
    dense, _ = dense_norm_adj(n, pairs.tolist())
    np.testing.assert_allclose(t.H_out, dense @ (H.astype(np.float64) @ W.astype(np.float64)),
                               rtol=2e-6, atol=1e-6)


def test_layer_is_the_l2_optimal_binary_approximation_chain():
    """General inputs: zeta must equal (beta F)(B alpha) as a dense float product of the two
    binarized approximations (Eq. "H-ip" / "cdot-op")."""
    rng = np.random.default_rng(23)
    n, d, c = 12, 37, 6
    pairs = random_pairs(rng, n, 30)
    g = oracle.normalize_adjacency(n, pairs[:, 0], pairs[:, 1])
    H = rng.standard_normal((n, d)).astype(np.float32)
    W = rng.standard_normal((d, c)).astype(np.float32)
    t = oracle.layer_forward(g, oracle.Layer(W), H)
    H_tilde = (np.abs(H).astype(np.float64).mean(1, keepdims=True)) * np.where(H >= 0, 1.0, -1.0)
    W_tilde = (np.abs(W).astype(np.float64).mean(0, keepdims=True)) * np.where(W >= 0, 1.0, -1.0)
    np.testing.assert_allclose(t.zeta, H_tilde @ W_tilde, rtol=1e-5, atol=1e-6)
    dense, _ = dense_norm_adj(n, pairs.tolist())
    np.testing.assert_allclose(t.H_out, dense @ (H_tilde @ W_tilde), rtol=1e-5, atol=1e-6)


def test_layer_from_packed_input_is_the_dense_product_of_its_own_input():
    """The layer that starts from an input that is already binary (packed signs and one scalar per node, Sec. 5.2):
    against the dense product A_tilde (diag(beta) F) (B diag(alpha)) formed with numpy from bits written by hand
    (np.packbits layout, not the oracle's packer), with beta an arbitrary vector that is NOT the row mean of
    anything; and equal, bit for bit, to the layer that binarizes the fp32 input itself when given that layer's bits."""
    rng = np.random.default_rng(24)
    n, d, c = 14, 45, 6
    pairs = random_pairs(rng, n, 35)
    g = oracle.normalize_adjacency(n, pairs[:, 0], pairs[:, 1])
    W = rng.standard_normal((d, c)).astype(np.float32)
    F = rng.choice(np.array([-1, 1], np.int8), size=(n, d))
    beta = (rng.random(n) * 2 + 0.1).astype(np.float32)
    stride = oracle.stride_words(d)
    padded = np.zeros((n, stride * 32), np.uint8)
    padded[:, :d] = F > 0
    bits = np.packbits(padded, axis=1, bitorder="little").view("<u4").reshape(n, stride)
    t = oracle.layer_forward_packed(g, oracle.Layer(W), bits, beta)
    alpha = np.abs(W).astype(np.float64).mean(0)
    dense, _ = dense_norm_adj(n, pairs.tolist())
    want = dense @ ((beta.astype(np.float64)[:, None] * F) @ (np.where(W >= 0, 1.0, -1.0) * alpha[None, :]))
    np.testing.assert_allclose(t.H_out, want, rtol=1e-5, atol=1e-6)
    assert np.array_equal(t.dot, F.astype(np.int64) @ np.where(W >= 0, 1, -1))
    # a transposed or mis-scaled operand would show: beta scales rows, alpha columns
    assert not np.allclose(t.H_out, dense @ ((F @ np.where(W >= 0, 1.0, -1.0)) * alpha[None, :]), rtol=1e-3)
    H = rng.standard_normal((n, d)).astype(np.float32)
    t1 = oracle.layer_forward(g, oracle.Layer(W), H)
    t2 = oracle.layer_forward_packed(g, oracle.Layer(W), t1.bits, t1.beta)
    assert np.array_equal(t1.H_out, t2.H_out) and np.array_equal(t1.dot, t2.dot) and np.array_equal(t1.zeta, t2.zeta)


def test_batchnorm_apply_balances_bits():
    rng = np.random.default_rng(31)
    H = (rng.random((400, 13)) < 0.05).astype(np.float32) * 3 + 2    # far from zero-centred
    shift, scale = oracle.col_stats(H)
    np.testing.assert_allclose(shift, H.mean(0), rtol=1e-6)
    np.testing.assert_allclose(scale, 1 / np.sqrt(H.astype(np.float64).var(0) + 1e-5), rtol=1e-6)
    xhat = (H - shift) * scale
    assert np.abs(xhat.mean(0)).max() < 1e-4 and np.abs(xhat.var(0) - 1).max() < 1e-3
    F, beta = oracle.binarize_rows(H, shift, scale)
    assert np.array_equal(F, np.where(xhat >= 0, 1, -1))
    np.testing.assert_allclose(beta, np.abs(xhat).mean(1), rtol=1e-6)
    F0, _ = oracle.binarize_rows(H)                                   # without it: all +1
    assert (F0 == 1).all()


def test_two_layer_forward_feeds_the_sign_of_the_first_output():
    rng = np.random.default_rng(41)
    n = 20
    pairs = random_pairs(rng, n, 50)
    g = oracle.normalize_adjacency(n, pairs[:, 0], pairs[:, 1])
    X = rng.standard_normal((n, 33)).astype(np.float32)
    W0 = rng.standard_normal((33, 8)).astype(np.float32)
    W1 = rng.standard_normal((8, 3)).astype(np.float32)
    logits, tr = oracle.forward(g, [oracle.Layer(W0), oracle.Layer(W1)], X)
    assert np.array_equal(tr[1].F, np.where(tr[0].H_out >= 0, 1, -1))   # no ReLU, sign acts
    assert np.array_equal(logits, tr[1].H_out) and logits.shape == (n, 3)


# ------------------------------------------------------------------ Sec. 5: the printed tables

def _golden_rows():
    rows = []
    for line in open(os.path.join(GOLDEN, "paper_cost_tables.txt")):
        line = line.strip()
        if line and not line.startswith("#"):
            name, n, e, dims, what, value, unit = line.split()
            rows.append((name, int(n), int(e), [int(x) for x in dims.split(",")], what, value, unit))
    return rows


@pytest.mark.parametrize("row", _golden_rows(), ids=lambda r: "%s-%s" % (r[0], r[4]))
def test_cost_model_reproduces_printed_tables(row):
    name, n, e, dims, what, value, unit = row
    got = oracle.cost_model(n, e, dims)[what]
    if unit == "exact":
        assert round(got) == int(value)
    elif unit == "sig3":
        printed = float(value)
        assert abs(got - printed) <= 0.006 * printed      # three significant digits
    else:
        scale = 1024.0 if unit[0] == "K" else 1024.0 ** 2
        digits = int(unit[1])
        assert abs(got / scale - float(value)) <= 0.5 * 10 ** (-digits) + 1e-9


def test_cost_model_ratios_of_table_1_and_sec_5_3():
    c = oracle.cost_model(2708, 5429, [1433, 64, 7])
    assert round(c["model_bytes_gcn"] / c["model_bytes_bigcn"], 1) == 31.2
    # Eq. "DC" gives 32 d / (d + 32) = 31.3 for d = 1433; the table's 31.5x is the ratio of its own
    # rounded entries 14.8M / 0.47M
    assert abs(c["data_bytes_gcn"] / c["data_bytes_bigcn"] - 32 * 1433 / (1433 + 32)) < 1e-9
    assert round(round(c["data_bytes_gcn"] / 2 ** 20, 1) / round(c["data_bytes_bigcn"] / 2 ** 20, 2), 1) == 31.5
    assert round(c["ops_gcn"] / c["ops_bigcn"], 1) == 53.5
    # per-layer feature-extraction speed-ups quoted in Sec. 5.3: ~59x and ~21x
    for d_in, quoted in ((1433, 59), (64, 21)):
        one = oracle.cost_model(1000, 0, [d_in, 16])
        assert round(one["ops_gcn"] / one["ops_bigcn"]) == quoted


# ------------------------------------------------------------------ Sec. 4.4.2: Bi-GraphSAGE

def test_mean_adjacency_rows_average_the_neighbours():
    rng = np.random.default_rng(61)
    n = 30
    pairs = random_pairs(rng, n, 60)
    pairs = np.concatenate([pairs, pairs[:10, ::-1], np.stack([np.arange(4)] * 2, 1).astype(np.int32)])
    keep = (pairs != 7).all(1)                       # node 7 stays isolated
    pairs = pairs[keep]
    g = oracle.mean_adjacency(n, pairs[:, 0], pairs[:, 1])
    A = np.zeros((n, n))
    for u, v in pairs.tolist():
        if u != v:
            A[u, v] = A[v, u] = 1.0
    deg = A.sum(1)
    M = to_dense(g)
    expect = np.divide(A, deg[:, None], out=np.zeros_like(A), where=deg[:, None] > 0)
    np.testing.assert_allclose(M, expect, rtol=1e-7, atol=0)
    assert M[7].sum() == 0 and g.rowptr[8] == g.rowptr[7]
    rows = M.sum(1)
    assert np.allclose(rows[deg > 0], 1.0, rtol=1e-6) and (np.diag(M) == 0).all()


def test_sage_layer_on_pm1_inputs_is_the_graphsage_mean_layer():
    """H, W_theta, W_n in {+-1}: scalars are 1 and the layer is W_theta h_i + mean_j W_n h_j exactly
    (Eq. "sage-conv" without the ReLU, which the binarized layer drops)."""
    rng = np.random.default_rng(62)
    n, d, c = 24, 37, 5
    pairs = random_pairs(rng, n, 50)
    g = oracle.mean_adjacency(n, pairs[:, 0], pairs[:, 1])
    H = rng.choice(np.array([-1.0, 1.0], np.float32), size=(n, d))
    Ws = rng.choice(np.array([-1.0, 1.0], np.float32), size=(d, c))
    Wn = rng.choice(np.array([-1.0, 1.0], np.float32), size=(d, c))
    t = oracle.sage_layer_forward(g, oracle.SageLayer(Ws, Wn), H)
    A = np.zeros((n, n))
    for u, v in pairs.tolist():
        if u != v:
            A[u, v] = A[v, u] = 1.0
    deg = A.sum(1)
    mean = np.divide(A, deg[:, None], out=np.zeros_like(A), where=deg[:, None] > 0)
    ref = H.astype(np.float64) @ Ws + mean @ (H.astype(np.float64) @ Wn)
    np.testing.assert_allclose(t.H_out, ref, rtol=1e-6, atol=1e-6)


def test_sage_layer_general_inputs_and_distinct_weights():
    """General inputs: the two terms use their own weights (a swap or a shared alpha would show)."""
    rng = np.random.default_rng(63)
    n, d, c = 15, 41, 6
    pairs = random_pairs(rng, n, 40)
    g = oracle.mean_adjacency(n, pairs[:, 0], pairs[:, 1])
    H = rng.standard_normal((n, d)).astype(np.float32)
    Ws = rng.standard_normal((d, c)).astype(np.float32)
    Wn = (3.0 * rng.standard_normal((d, c))).astype(np.float32)
    t = oracle.sage_layer_forward(g, oracle.SageLayer(Ws, Wn), H)
    Ht = np.abs(H).astype(np.float64).mean(1, keepdims=True) * np.where(H >= 0, 1.0, -1.0)
    Wst = np.abs(Ws).astype(np.float64).mean(0, keepdims=True) * np.where(Ws >= 0, 1.0, -1.0)
    Wnt = np.abs(Wn).astype(np.float64).mean(0, keepdims=True) * np.where(Wn >= 0, 1.0, -1.0)
    ref = Ht @ Wst + to_dense(g) @ (Ht @ Wnt)
    np.testing.assert_allclose(t.H_out, ref, rtol=1e-5, atol=1e-6)


# --------------------------------------------------------------------------- entropy estimator (Sec. 6.2)

def test_entropy_uniform_column_is_log2_of_the_interval_count():
    """N = r * M samples spread evenly over the range fill every interval r times: H = log2 M exactly."""
    M, r = 64, 5
    x = np.repeat(np.arange(M, dtype=np.float32) + 0.5, r)        # r samples in the middle of each unit interval
    x = np.concatenate([x, np.float32([0.0, M])])                  # pin the range to [0, M]: +1 in the first and last
    rng = np.random.default_rng(1)
    H = rng.permutation(x)[:, None].astype(np.float32)
    est = oracle.entropy_bins(H, M)
    assert est.col_min[0] == 0.0 and est.col_max[0] == M
    want = np.full(M, r); want[0] += 1; want[-1] += 1              # the maximum falls into the last interval
    assert np.array_equal(est.counts[0], want)
    p = want / want.sum()
    assert est.entropy[0] == pytest.approx(-(p * np.log2(p)).sum(), rel=1e-14)
    assert est.entropy[0] == pytest.approx(np.log2(M), abs=2e-3) and est.entropy[0] < np.log2(M)


def test_entropy_closed_forms():
    n = 1000
    H = np.zeros((n, 4), np.float32)
    H[:, 0] = 3.25                                                 # constant neuron: no information
    H[: n // 2, 1] = -1.0; H[n // 2:, 1] = 2.0                     # fair coin: one bit
    H[: n // 4, 2] = 0.0; H[n // 4:, 2] = 1.0                      # 1/4 - 3/4 split
    H[:, 3] = np.arange(n, dtype=np.float32)                       # n distinct values, M >= n intervals: log2 n bits
    est = oracle.entropy_bins(H, 4096)
    assert est.entropy[0] == 0.0 and est.counts[0, 0] == n and est.counts[0, 1:].sum() == 0
    assert est.entropy[1] == pytest.approx(1.0, abs=1e-15)
    assert est.entropy[2] == pytest.approx(-(0.25 * np.log2(0.25) + 0.75 * np.log2(0.75)), rel=1e-14)
    assert est.entropy[3] == pytest.approx(np.log2(n), rel=1e-12)
    assert est.total == pytest.approx(est.entropy.sum(), rel=1e-15)   # H_ind is the plain sum over the neurons
    assert (est.counts.sum(axis=1) == n).all()


def test_entropy_against_library_histogram():
    """numpy's histogram over the same M equal-width intervals of [min, max] is the same empirical
    distribution (up to samples that sit on an interval edge to within fp32 rounding)."""
    rng = np.random.default_rng(7)
    n, d, M = 20000, 6, 200
    H = (rng.standard_normal((n, d)) * rng.uniform(0.5, 3.0, d) + rng.uniform(-2, 2, d)).astype(np.float32)
    H[:, 1] = np.maximum(H[:, 1], 0)                               # a rectified neuron: a spike in the first interval
    est = oracle.entropy_bins(H, M)
    for j in range(d):
        c, _ = np.histogram(H[:, j].astype(np.float64), bins=M, range=(float(H[:, j].min()), float(H[:, j].max())))
        assert np.abs(c - est.counts[j]).sum() <= 8                # edge cases only
        p = c[c > 0] / n
        assert est.entropy[j] == pytest.approx(-(p * np.log2(p)).sum(), abs=2e-3)
        assert est.entropy[j] <= np.log2(M)
    assert est.col_min.tolist() == H.min(axis=0).tolist() and est.col_max.tolist() == H.max(axis=0).tolist()


def test_entropy_permutation_and_affine_invariance():
    """The estimate depends on the empirical distribution only: the order of the samples does not matter,
    and a power-of-two rescaling plus shift of a neuron (exact in fp32 here) leaves every count unchanged."""
    rng = np.random.default_rng(11)
    H = np.round(rng.standard_normal((5000, 3)) * 64).astype(np.float32)     # multiples of 1: shifts stay exact
    a = oracle.entropy_bins(H, 100)
    b = oracle.entropy_bins(H[rng.permutation(len(H))], 100)
    c = oracle.entropy_bins(H * np.float32(4.0) + np.float32(1024.0), 100)
    assert np.array_equal(a.counts, b.counts) and np.array_equal(a.counts, c.counts)
    assert np.array_equal(a.entropy, b.entropy) and np.array_equal(a.entropy, c.entropy)


def test_entropy_table_of_the_paper_fixes_the_logarithm():
    """Every printed estimate respects H <= n_h log2 M; the PubMed one exceeds n_h ln M, so the paper's
    logarithm cannot be the natural one: bits."""
    rows = [l.split() for l in open(os.path.join(GOLDEN, "paper_entropy_table.txt")) if l.strip() and not l.startswith("#")]
    assert len(rows) == 4
    for name, kind, nh, ns, M, h in rows:
        nh, ns, M, h = int(nh), int(ns), int(M), float(h)
        assert h <= nh * np.log2(M)
        assert h <= nh * np.log2(ns)
    nh, M, h = int(rows[0][2]), int(rows[0][4]), float(rows[0][5])
    assert h > nh * np.log(M)
    # and the oracle attains the bound it is held to: M equally likely intervals give log2 M per neuron
    x = (np.arange(M * 3, dtype=np.float32) % M)[:, None]
    est = oracle.entropy_bins(np.concatenate([x, np.float32([[M]])]), M)
    assert est.entropy[0] == pytest.approx(np.log2(M), abs=1e-2)


# --------------------------------------------------------------------------- back-propagation (Algorithm 1)

def _bw_case(seed, n=23, d_in=11, d_out=7, asym=False):
    rng = np.random.default_rng(seed)
    src = rng.integers(0, n, 3 * n); dst = rng.integers(0, n, 3 * n)
    g = oracle.normalize_adjacency(n, src, dst)
    if asym:                                   # a non-symmetric sparse matrix on the same pattern: tells A^T from A
        g = oracle.Graph(g.n, g.rowptr, g.colidx, (g.val * rng.uniform(0.5, 1.5, g.val.shape)).astype(np.float32), g.dinv)
    W = (rng.standard_normal((d_in, d_out)) * 0.8).astype(np.float32)
    H = rng.standard_normal((n, d_in)).astype(np.float32)
    F, beta = oracle.binarize_rows(H)
    G = (rng.standard_normal((n, d_out)) * 0.3).astype(np.float32)
    return g, W, F, beta, G


def _dense(g):
    A = np.zeros((g.n, g.n))
    for i in range(g.n):
        for e in range(g.rowptr[i], g.rowptr[i + 1]):
            A[i, g.colidx[e]] += float(g.val[e])
    return A


def test_backward_step1_is_the_gradient_of_the_linear_forward():
    """H' = A (H~ W~) is linear in H~ and in W~: with L = <G', H'> the gradients are A^T G', H~^T A^T G' and
    A^T G' W~^T exactly.  Checked against dense matrix algebra on a NON-symmetric A (so that A and A^T, and
    every other transposition, cannot be confused) and against central differences of the dense forward."""
    g, W, F, beta, G = _bw_case(1, asym=True)
    bw = oracle.layer_backward(g, W, F, beta, G)
    A = _dense(g)
    Bm, alpha = oracle.binarize_cols(W)
    Ht = beta[:, None].astype(np.float64) * F
    Wt = alpha[None, :].astype(np.float64) * Bm
    Gz = A.T @ G.astype(np.float64)
    np.testing.assert_allclose(bw.G_zeta, Gz, rtol=1e-6, atol=1e-7)
    np.testing.assert_allclose(bw.G_Wt, Ht.T @ Gz, rtol=1e-6, atol=1e-6)
    np.testing.assert_allclose(bw.G_Ht, Gz @ Wt.T, rtol=1e-6, atol=1e-6)
    assert not np.allclose(bw.G_zeta, A @ G, rtol=1e-3, atol=1e-4)          # the untransposed product is different
    loss = lambda Hx, Wx: float((G.astype(np.float64) * (A @ (Hx @ Wx))).sum())
    rng = np.random.default_rng(2)
    for _ in range(6):
        i, k, j = rng.integers(g.n), rng.integers(W.shape[0]), rng.integers(W.shape[1])
        E = np.zeros_like(Wt); E[k, j] = 1.0
        assert (loss(Ht, Wt + E) - loss(Ht, Wt - E)) / 2 == pytest.approx(bw.G_Wt[k, j], rel=1e-5, abs=1e-6)
        E = np.zeros_like(Ht); E[i, k] = 1.0
        assert (loss(Ht + E, Wt) - loss(Ht - E, Wt)) / 2 == pytest.approx(bw.G_Ht[i, k], rel=1e-5, abs=1e-6)


def test_backward_eq_bp_H_is_a_strict_clip():
    g, W, F, beta, G = _bw_case(3)
    bw = oracle.layer_backward(g, W, F, beta, G * 8)                      # large enough that some |G_H~| exceed 1
    big = np.abs(bw.G_Ht) >= 1
    assert big.any() and (~big).any()
    assert (bw.G_H[big] == 0).all() and np.array_equal(bw.G_H[~big], bw.G_Ht[~big])
    # the boundary itself is excluded (|r| < 1): one node, one feature, weight 1, gradient exactly 1
    g1 = oracle.Graph(1, np.array([0, 1], np.int64), np.array([0], np.int32), np.array([1.0], np.float32), np.ones(1, np.float32))
    one = oracle.layer_backward(g1, np.array([[1.0]], np.float32), np.array([[1]], np.int8), np.ones(1, np.float32), np.array([[1.0]], np.float32))
    assert one.G_Ht[0, 0] == 1.0 and one.G_H[0, 0] == 0.0
    half = oracle.layer_backward(g1, np.array([[1.0]], np.float32), np.array([[1]], np.int8), np.ones(1, np.float32), np.array([[0.5]], np.float32))
    assert half.G_H[0, 0] == 0.5


def test_backward_eq_bp_W_terms():
    """First term: the derivative through alpha_j = ||W_:,j||_1 / d_in with the signs held fixed, checked by
    central differences.  Second term: alpha_j G_W~_ij where |W_ij| < 1 (straight-through estimate), else 0."""
    g, W, F, beta, G = _bw_case(5)
    W[0, 0] = 1.5; W[1, 0] = -1.0; W[2, 0] = 0.999                        # outside, on and inside the STE window
    bw = oracle.layer_backward(g, W, F, beta, G)
    Bm, alpha = oracle.binarize_cols(W)
    d_in = W.shape[0]
    col = (bw.G_Wt.astype(np.float64) * Bm).sum(axis=0)
    first = Bm * col[None, :] / d_in
    second = np.where(np.abs(W) < 1, alpha[None, :].astype(np.float64) * bw.G_Wt, 0.0)
    # (G_W~ is read back rounded to fp32 here, the oracle carries it in double: 1e-5)
    np.testing.assert_allclose(bw.G_W, first + second, rtol=1e-5, atol=1e-7)
    assert bw.G_W[0, 0] == pytest.approx(first[0, 0], rel=1e-5) and bw.G_W[1, 0] == pytest.approx(first[1, 0], rel=1e-5)
    assert bw.G_W[2, 0] == pytest.approx(first[2, 0] + alpha[0] * bw.G_Wt[2, 0], rel=1e-5)
    # finite differences of L(W) = <G_W~, alpha(W) B> with B fixed reproduce the first term
    Gwt = bw.G_Wt.astype(np.float64)
    L = lambda Wx: float((Gwt * (np.abs(Wx).sum(axis=0, keepdims=True) / d_in * Bm)).sum())
    for (i, j) in [(0, 0), (3, 2), (7, 6)]:
        h = 1e-3
        E = np.zeros(W.shape); E[i, j] = h
        Wd = W.astype(np.float64)
        assert (L(Wd + E) - L(Wd - E)) / (2 * h) == pytest.approx(first[i, j], rel=1e-6, abs=1e-9)


def test_backward_plain_gcn_special_case():
    """With +-1 inputs and +-1 weights (beta = alpha = 1) the layer is the plain GCN layer A X W, whose
    gradients are textbook: dL/dW = X^T A^T G', dL/dX = A^T G' W^T."""
    rng = np.random.default_rng(9)
    n, d_in, d_out = 15, 6, 4
    g = oracle.normalize_adjacency(n, rng.integers(0, n, 30), rng.integers(0, n, 30))
    X = rng.choice([-1.0, 1.0], (n, d_in)).astype(np.float32)
    W = rng.choice([-1.0, 1.0], (d_in, d_out)).astype(np.float32)
    F, beta = oracle.binarize_rows(X)
    assert (beta == 1).all()
    G = (rng.standard_normal((n, d_out)) * 0.01).astype(np.float32)
    bw = oracle.layer_backward(g, W, F, beta, G)
    A = _dense(g)
    np.testing.assert_allclose(bw.G_Wt, X.T.astype(np.float64) @ A.T @ G, rtol=1e-6, atol=1e-8)
    np.testing.assert_allclose(bw.G_H, A.T @ G.astype(np.float64) @ W.T, rtol=1e-6, atol=1e-8)   # all |.| < 1: no clipping
    # |W_ij| = 1 is outside the STE window: only the alpha-path term of Eq. bp-W remains
    col = (bw.G_Wt.astype(np.float64) * W).sum(axis=0)
    np.testing.assert_allclose(bw.G_W, W * col[None, :] / d_in, rtol=1e-5, atol=1e-9)

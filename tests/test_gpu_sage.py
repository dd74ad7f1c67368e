"""GPU parity of the Bi-GraphSAGE layer (Sec. 4.4.2, Eq. "bisage-conv") against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2210_13149_b200 import synth
from parity_util import ATOL, RTOL, assert_close, bits_from_dev, bits_to_dev, dev, flip_report

pytestmark = pytest.mark.gpu


@pytest.fixture()
def ctx():
    from paper_2210_13149_b200 import binding
    c = binding.BiGCN(0)
    yield c
    c.sync_check()
    c.close()


@pytest.mark.parametrize("n,e,seed", [(1, 0, 1), (9, 0, 2), (60, 300, 3), (3327, 9104, 1002), (4000, 300000, 5)])
def test_mean_adjacency_is_bit_exact(ctx, n, e, seed):
    rp, ci = synth.power_law_graph(n, e, seed)
    src, dst = synth.edge_list(rp, ci)
    g = oracle.mean_adjacency(n, src, dst)
    got = ctx.mean_adjacency(rp.cuda(), ci.cuda())
    assert got.nnz == g.nnz
    assert np.array_equal(got.rowptr.cpu().numpy(), g.rowptr)
    assert np.array_equal(got.colidx.cpu().numpy(), g.colidx)
    assert np.array_equal(got.val.cpu().numpy(), g.val)
    assert np.array_equal(got.dinv.cpu().numpy(), g.dinv)


# storage of the neighbours' dots between contraction and aggregation: 0 = the automatic choice (bytes for 129..256
# columns when d_in <= 127), 1 fp32, 2 int16, 3 bytes, 4 fp16, 5 half-dot bytes (not offered to this layer: falls back);
# the (4200, .., 256, 256) case has 2^20 outputs, from where the contraction runs on the tensor cores
@pytest.mark.parametrize("fmt", [0, 1, 2, 3, 4, 5])
@pytest.mark.parametrize("n,e,d_in,d_out", [(300, 2500, 33, 7), (500, 6000, 100, 256), (400, 5000, 602, 256),
                                             (600, 9000, 256, 47), (450, 4000, 64, 6), (350, 3000, 1433, 64),
                                             (4200, 50000, 256, 256)])
def test_sage_layer_against_oracle(ctx, fmt, n, e, d_in, d_out):
    check_sage_layer(ctx, fmt, n, e, d_in, d_out)


@pytest.mark.parametrize("n,e,d_in,d_out", [(500, 6000, 100, 256), (300, 200, 64, 200), (4200, 50000, 127, 256)])
def test_sage_layer_with_the_tensor_core_aggregation(ctx, n, e, d_in, d_out):
    """The neighbours' term as tcgen05 integer products (byte rows of 129..256 columns); the second shape has
    mostly isolated nodes, whose rows of the mean aggregator are empty and must come out as the node's own term."""
    from paper_2210_13149_b200 import binding as B
    ctx.set_option(B.OPT_BYTE_AGGREGATION, 3)
    try:
        check_sage_layer(ctx, 0, n, e, d_in, d_out)
    finally:
        ctx.set_option(B.OPT_BYTE_AGGREGATION, 0)


def check_sage_layer(ctx, fmt, n, e, d_in, d_out):
    from paper_2210_13149_b200 import binding as B
    rng = np.random.default_rng(n + 5 * d_in + 11 * d_out)
    rp, ci = synth.power_law_graph(n, e, 200 + n)
    src, dst = synth.edge_list(rp, ci)
    g = oracle.mean_adjacency(n, src, dst)
    H = rng.standard_normal((n, d_in)).astype(np.float32)
    Ws = (rng.standard_normal((d_in, d_out)) * d_in ** -0.5).astype(np.float32)
    Wn = (rng.standard_normal((d_in, d_out)) * 2 * d_in ** -0.5).astype(np.float32)
    t = oracle.sage_layer_forward(g, oracle.SageLayer(Ws, Wn), H)
    nshift, nscale = oracle.col_stats(t.H_out)
    Fn, beta_n = oracle.binarize_rows(t.H_out, nshift, nscale)

    ctx.set_option(B.OPT_ZETA_FORMAT, fmt)
    G = B.make_graph(dev(g.rowptr), dev(g.colidx), dev(g.val), dev(g.dinv))
    ls = B.make_layer(d_in, d_out, bits_to_dev(t.bitsT_self), dev(t.alpha_self))
    ln = B.make_layer(d_in, d_out, bits_to_dev(t.bitsT_nbr), dev(t.alpha_nbr))
    dummy = torch.zeros((4, B.packed_stride_words(d_out)), dtype=torch.int32).cuda()
    nxt = B.make_layer(d_out, 4, dummy, torch.ones(4).cuda(), dev(nshift), dev(nscale))
    out = ctx.sage_layer_forward(G, ls, ln, bits_to_dev(t.bits), dev(t.beta), want_h=True, next_layer=nxt)
    assert_close(out["h"], t.H_out, "Bi-GraphSAGE layer output")
    flips, bad, total = flip_report(bits_from_dev(out["next_bits"]), Fn, t.H_out, nshift)
    assert bad == 0 and flips <= max(2, total // 2000), (flips, bad, total)
    np.testing.assert_allclose(out["next_beta"].cpu().numpy(), beta_n, rtol=RTOL, atol=ATOL)


def test_sage_layer_on_pm1_inputs_is_the_graphsage_mean_layer(ctx):
    from paper_2210_13149_b200 import binding as B
    rng = np.random.default_rng(64)
    n, d, c = 200, 45, 5
    rp, ci = synth.power_law_graph(n, 1200, 64)
    G = ctx.mean_adjacency(rp.cuda(), ci.cuda())
    H = rng.choice(np.array([-1.0, 1.0], np.float32), size=(n, d))
    Ws = rng.choice(np.array([-1.0, 1.0], np.float32), size=(d, c))
    Wn = rng.choice(np.array([-1.0, 1.0], np.float32), size=(d, c))
    bits, beta = ctx.pack_features(dev(H))
    bs, a_s = ctx.pack_weights(dev(Ws))
    bn, a_n = ctx.pack_weights(dev(Wn))
    out = ctx.sage_layer_forward(G, B.make_layer(d, c, bs, a_s), B.make_layer(d, c, bn, a_n), bits, beta)
    A = torch.sparse_csr_tensor(G.rowptr, G.colidx.long(), G.val.double(), size=(n, n)).to_dense()
    ref = dev(H).double() @ dev(Ws).double() + A @ (dev(H).double() @ dev(Wn).double())
    assert_close(out["h"], ref.float().cpu(), "GraphSAGE special case")


def test_two_sage_layers_chain_through_the_fused_rebinarization(ctx):
    from paper_2210_13149_b200 import binding as B
    rng = np.random.default_rng(65)
    n, dims = 1500, [100, 64, 7]
    rp, ci = synth.power_law_graph(n, 20000, 65)
    src, dst = synth.edge_list(rp, ci)
    g = oracle.mean_adjacency(n, src, dst)
    X = rng.standard_normal((n, dims[0])).astype(np.float32)
    W = [[(rng.standard_normal((a, b)) * a ** -0.5).astype(np.float32) for _ in range(2)] for a, b in zip(dims[:-1], dims[1:])]
    sh0, sc0 = oracle.col_stats(X)
    t0 = oracle.sage_layer_forward(g, oracle.SageLayer(W[0][0], W[0][1], sh0, sc0), X)
    t1 = oracle.sage_layer_forward(g, oracle.SageLayer(W[1][0], W[1][1]), t0.H_out)
    G = ctx.mean_adjacency(rp.cuda(), ci.cuda())
    layers = []
    for (Ws, Wn), (a, b) in zip(W, zip(dims[:-1], dims[1:])):
        bs, a_s = ctx.pack_weights(dev(Ws))
        bn, a_n = ctx.pack_weights(dev(Wn))
        layers.append((B.make_layer(a, b, bs, a_s), B.make_layer(a, b, bn, a_n)))
    bits, beta = ctx.pack_features(dev(X), dev(sh0), dev(sc0))
    assert np.array_equal(bits_from_dev(bits), t0.bits)
    o0 = ctx.sage_layer_forward(G, layers[0][0], layers[0][1], bits, beta, want_h=True, next_layer=layers[1][0])
    assert_close(o0["h"], t0.H_out, "layer 0")
    # the re-binarized bits differ from the oracle's only at the threshold
    flips, bad, total = flip_report(bits_from_dev(o0["next_bits"]), t1.F, t0.H_out, None)
    assert bad == 0 and flips <= 4, (flips, bad, total)
    o1 = ctx.sage_layer_forward(G, layers[1][0], layers[1][1], o0["next_bits"], o0["next_beta"], want_h=True)
    # every row of the second layer against the oracle's steps on the very input it saw (the GPU's own bits and beta)
    own_bits, own_beta = bits_from_dev(o0["next_bits"]), o0["next_beta"].cpu().numpy()
    Bs, a_s = oracle.binarize_cols(W[1][0])
    Bn, a_n = oracle.binarize_cols(W[1][1])
    z_s = oracle.rescale(oracle.dot_popc(own_bits, oracle.pack_cols(Bs), dims[1]), own_beta, a_s)
    z_n = oracle.rescale(oracle.dot_popc(own_bits, oracle.pack_cols(Bn), dims[1]), own_beta, a_n)
    assert_close(o1["h"], oracle.spmm_add(g, z_n, z_s), "logits on the GPU's own second-layer input")
    if flips == 0:
        assert_close(o1["h"], t1.H_out, "logits")

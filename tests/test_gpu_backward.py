"""bigcn_layer_backward against the oracle's Algorithm 1 (Sec. 4.3, Eq. bp-H, Eq. bp-W).

The oracle sums in double, the GPU in fp32 (sums over the nodes in slabs added in a fixed order).
Tolerance, from that arithmetic: |got - ref| <= 1e-4 |ref| + 2e-6 max|ref| (a sum of m terms in fp32
carries about sqrt(m) * 6e-8 of the largest partial sum).  Eq. bp-H decides 0-or-pass by |G_H~| < 1:
an element whose reference |G_H~| lies within the tolerance of 1 may fall on either side.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2210_13149_b200 import synth
from parity_util import bits_to_dev, dev, device_graph

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2210_13149_b200 import binding
    return binding


@pytest.fixture(scope="module")
def ctx(B):
    c = B.BiGCN(0)
    yield c
    c.close()


def close(got, ref, what):
    got = got.cpu().numpy().astype(np.float64)
    ref = ref.astype(np.float64)
    allow = 1e-4 * np.abs(ref) + 2e-6 * max(np.abs(ref).max(), 1e-30)
    bad = np.abs(got - ref) > allow
    assert not bad.any(), "%s: %d of %d outside tolerance, worst %.3g" % (what, bad.sum(), bad.size, (np.abs(got - ref) / allow).max())


def run_case(B, ctx, n, m, d_in, d_out, seed, g_scale=0.05, want_g_in=True, w_scale=0.8):
    rng = np.random.default_rng(seed)
    g = oracle.normalize_adjacency(n, rng.integers(0, n, m), rng.integers(0, n, m))
    W = (rng.standard_normal((d_in, d_out)) * w_scale).astype(np.float32)
    H = rng.standard_normal((n, d_in)).astype(np.float32)
    F, beta = oracle.binarize_rows(H)
    G_out = (rng.standard_normal((n, d_out)) * g_scale).astype(np.float32)
    ref = oracle.layer_backward(g, W, F, beta, G_out)

    G = device_graph(B, g)
    Wd = dev(W)
    bitsT, alpha = ctx.pack_weights(Wd)
    layer = B.make_layer(d_in, d_out, bitsT, alpha)
    bits = bits_to_dev(oracle.pack_rows(F))          # both sides get the oracle's bits and row scales
    beta_d = dev(beta)
    g_in, g_w = ctx.layer_backward(G, layer, Wd, bits, beta_d, dev(G_out), want_g_in=want_g_in)
    ctx.sync_check()
    close(g_w, ref.G_W, "G_W")
    if want_g_in:
        got = g_in.cpu().numpy()
        near = np.abs(np.abs(ref.G_Ht.astype(np.float64)) - 1.0) <= 2e-4          # the clip may go either way here
        exact = ~near
        close(torch.from_numpy(np.where(exact, got, 0)), np.where(exact, ref.G_H, 0), "G_H")
        on_edge = got[near]
        assert np.all((on_edge == 0) | (np.abs(on_edge - ref.G_Ht[near]) <= 2e-4))
        clipped = (np.abs(ref.G_Ht) >= 1).mean()
    else:
        assert g_in is None
        clipped = None
    return ref, clipped


@pytest.mark.parametrize("n,m,d_in,d_out", [(1, 0, 1, 1), (23, 60, 11, 7), (300, 2000, 100, 256), (500, 3000, 256, 47),
                                            (1000, 6000, 64, 64), (777, 5000, 130, 200), (2000, 30000, 256, 256),
                                            (400, 3000, 300, 40), (129, 700, 128, 130), (20000, 100000, 256, 256)])   # d_in > 256: the mma.sync kernels; several chunks and tiles per CTA
def test_backward_matches_oracle(B, ctx, n, m, d_in, d_out):
    run_case(B, ctx, n, m, d_in, d_out, seed=n + d_in)


def test_backward_clip_is_exercised(B, ctx):
    """Upstream gradients large enough that a good share of |G_H~| exceeds 1: those elements must be 0."""
    ref, clipped = run_case(B, ctx, 400, 4000, 64, 32, seed=5, g_scale=3.0)
    assert 0.05 < clipped < 0.95
    assert (ref.G_H[np.abs(ref.G_Ht) >= 1] == 0).all()


def test_backward_ste_window_is_exercised(B, ctx):
    """Weights on both sides of |W| = 1: the straight-through term is present for some and absent for others."""
    rng = np.random.default_rng(8)
    ref, _ = run_case(B, ctx, 350, 2500, 48, 40, seed=8, w_scale=1.2)


def test_backward_first_layer_needs_no_input_gradient(B, ctx):
    run_case(B, ctx, 600, 4000, 1433, 64, seed=2, want_g_in=False)


def test_backward_on_a_workload_layer(B, ctx):
    """Layer 1 of c3 (hidden -> classes) with its real forward input: the packed output of layer 0."""
    wl = synth.make_workload("c3", device="cuda")
    Gd = ctx.normalize_adjacency(wl.rowptr.cuda(), wl.colidx.cuda())
    layers = ctx.prepare_layers([w.cuda() for w in wl.W])
    xb, xbeta = ctx.pack_features(wl.X.cuda())
    out = ctx.layer_forward(Gd, layers[0], xb, xbeta, next_layer=layers[1])
    bits1, beta1 = out["next_bits"], out["next_beta"]
    n, d_in, d_out = wl.n, layers[1].d_in, layers[1].d_out
    gen = torch.Generator(device="cuda").manual_seed(4)
    g_out = torch.randn((n, d_out), device="cuda", generator=gen) * 0.02
    g_in, g_w = ctx.layer_backward(Gd, layers[1], wl.W[1].cuda(), bits1, beta1, g_out)
    # the oracle on the same inputs (bits unpacked on the host)
    src, dst = synth.edge_list(wl.rowptr, wl.colidx)
    g = oracle.normalize_adjacency(n, src, dst)
    F = oracle.unpack_rows(bits1.cpu().numpy().view(np.uint32), d_in)
    ref = oracle.layer_backward(g, wl.W[1].cpu().numpy(), F, beta1.cpu().numpy(), g_out.cpu().numpy())
    close(g_w, ref.G_W, "G_W (c3 layer 1)")
    near = np.abs(np.abs(ref.G_Ht.astype(np.float64)) - 1.0) <= 2e-4
    close(torch.from_numpy(np.where(~near, g_in.cpu().numpy(), 0)), np.where(~near, ref.G_H, 0), "G_H (c3 layer 1)")


def test_backward_argument_checks(B, ctx):
    import ctypes
    rng = np.random.default_rng(1)
    g = oracle.normalize_adjacency(10, rng.integers(0, 10, 20), rng.integers(0, 10, 20))
    G = device_graph(B, g)
    W = torch.randn((8, 600), device="cuda")
    bitsT, alpha = ctx.pack_weights(W)
    layer = B.make_layer(8, 600, bitsT, alpha)
    bits, beta = ctx.pack_features(torch.randn((10, 8), device="cuda"))
    before = ctx.launch_count()
    with pytest.raises(B.BigcnError) as e:
        ctx.layer_backward(G, layer, W, bits, beta, torch.zeros((10, 600), device="cuda"))
    assert e.value.status == 7 and ctx.launch_count() == before                 # d_out > 512
    assert ctx.lib.bigcn_backward_workspace_bytes(1000, 64, 64) >= 2 * 1000 * 64 * 4
    ctx.sync_check()

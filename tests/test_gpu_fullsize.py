"""GPU parity at the full size of the two large configurations, in the launch configuration the
benchmark times.  The oracle runs the whole forward once on the host cores (tens of seconds); every
element of every layer is then compared on the device."""
import numpy as np
import pytest
import torch

import oracle
from paper_2210_13149_b200 import synth
from parity_util import (ATOL, RTOL, bits_to_dev, dev, device_layers_from_oracle, end_to_end_with_flip_accounting,
                         oracle_run, unpack_signs_dev, within_tol)

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["c4", "c5"])
def test_full_size_layers_oracle_fed_and_end_to_end(name):
    from paper_2210_13149_b200 import binding as B
    wl = synth.make_workload(name, device="cuda")
    run = oracle_run(wl, keep_trace=True)
    ctx = B.BiGCN(0)
    G = ctx.normalize_adjacency(wl.rowptr.cuda(), wl.colidx.cuda())
    # the set-up step at full size: structure and values bit for bit
    assert G.nnz == run.graph.nnz
    assert torch.equal(G.rowptr.cpu(), torch.from_numpy(run.graph.rowptr))
    assert torch.equal(G.colidx.cpu(), torch.from_numpy(run.graph.colidx))
    assert torch.equal(G.val.cpu(), torch.from_numpy(run.graph.val))
    layers = device_layers_from_oracle(B, run)
    L = len(layers)
    for l in range(L):
        t = run.traces[l]
        nxt = layers[l + 1] if l + 1 < L else None
        out = ctx.layer_forward(G, layers[l], bits_to_dev(t.bits), dev(t.beta), want_h=True, next_layer=nxt, debug=True)
        assert torch.equal(out["dot"], dev(t.dot)), "layer %d: integer dot products differ" % l
        assert torch.equal(out["zeta"], dev(t.zeta)), "layer %d: zeta differs" % l
        ok, ratio, mx = within_tol(out["h"], torch.from_numpy(t.H_out))
        assert ok, "layer %d: H' error / allowance = %.3g (max abs %.3g)" % (l, ratio, mx)
        if nxt is not None:
            tn = run.traces[l + 1]
            got = unpack_signs_dev(out["next_bits"], layers[l].d_out)
            ref = dev(tn.F) > 0
            diff = got != ref
            H = dev(t.H_out).double()
            mu = dev(run.layers[l + 1].in_shift).double() if run.layers[l + 1].in_shift is not None else 0.0
            near = (H - mu).abs() <= ATOL + RTOL * H.abs()
            flips, bad = int(diff.sum()), int((diff & ~near).sum())
            print("\n[%s] layer %d: %d re-binarized bits of %d differ, %d away from the threshold" % (name, l, flips, diff.numel(), bad))
            assert bad == 0 and flips <= diff.numel() // 100000 + 2
            del got, ref, diff, H, near
        del out
    # end to end through the library's own packers, in the benchmark's launch configuration
    shifts = [dev(x.in_shift) if x.in_shift is not None else None for x in run.layers]
    scales = [dev(x.in_scale) if x.in_scale is not None else None for x in run.layers]
    own = ctx.prepare_layers([w.cuda() for w in wl.W], shifts, scales)
    X = wl.X.cuda()
    rep = end_to_end_with_flip_accounting(ctx, G, own, run, X)
    print("[%s] end to end: %s" % (name, rep))
    assert rep["argmax_agreement"] >= 0.995
    assert sum(rep["origin_flips"]) <= 100
    # the one-call forward gives the same logits as the layer-by-layer run just checked
    logits = ctx.forward(G, own, X)
    last = own[-1]
    ref = dev(run.logits)
    err = (logits.double() - ref.double()).abs()
    share_out = float((err > ATOL + RTOL * ref.double().abs()).double().mean())
    assert abs(share_out - rep["logits_outside_tolerance"]) < 1e-12
    ctx.sync_check()
    ctx.close()


def test_entropy_bins_full_size():
    """The side benchmark's configuration (the largest row of the paper's entropy table: 2,449,029 samples x 128
    neurons, 1000 intervals): every count against the oracle's."""
    import oracle
    n, d, M = 2449029, 128, 1000
    g = torch.Generator(device="cuda").manual_seed(2210)
    H = torch.randn((n, d), device="cuda", generator=g) * (torch.rand(d, device="cuda", generator=g) * 3.8 + 0.2)
    H[:, ::4].clamp_(min=0)
    from paper_2210_13149_b200 import binding
    ctx = binding.BiGCN(0)
    got = ctx.entropy_bins(H, M)
    want = oracle.entropy_bins(H.cpu().numpy(), M)
    assert np.array_equal(got["col_min"].cpu().numpy(), want.col_min)
    assert np.array_equal(got["col_max"].cpu().numpy(), want.col_max)
    assert np.array_equal(got["counts"].cpu().numpy().astype(np.int64), want.counts)
    np.testing.assert_allclose(got["entropy"].cpu().numpy(), want.entropy, rtol=1e-12)
    assert got["total"].item() == pytest.approx(want.total, rel=1e-12)
    ctx.close()


def test_backward_large_graph_sampled_rows():
    """Algorithm 1 on the c5 recipe at a twentieth of its size (122 k nodes, 6 M entries), 256 -> 64: the weight
    gradient (a sum over every node) in full, the input gradient on every row."""
    import oracle
    from paper_2210_13149_b200 import binding, synth
    wl = synth.make_workload("c5", scale=0.05, device="cuda")
    n, d_in, d_out = wl.n, 256, 64
    ctx = binding.BiGCN(0)
    G = ctx.normalize_adjacency(wl.rowptr, wl.colidx)
    gen = torch.Generator(device="cuda").manual_seed(5)
    W = torch.randn((d_in, d_out), device="cuda", generator=gen) * 0.7
    Hin = torch.randn((n, d_in), device="cuda", generator=gen)
    g_out = torch.randn((n, d_out), device="cuda", generator=gen) * 0.02
    bitsT, alpha = ctx.pack_weights(W)
    layer = binding.make_layer(d_in, d_out, bitsT, alpha)
    bits, beta = ctx.pack_features(Hin)
    g_in, g_w = ctx.layer_backward(G, layer, W, bits, beta, g_out)
    src, dst = synth.edge_list(wl.rowptr, wl.colidx)
    g = oracle.normalize_adjacency(n, src, dst)
    F = oracle.unpack_rows(bits.cpu().numpy().view(np.uint32), d_in)
    ref = oracle.layer_backward(g, W.cpu().numpy(), F, beta.cpu().numpy(), g_out.cpu().numpy())

    def close(got, want, what):
        got = got.astype(np.float64); want = want.astype(np.float64)
        allow = 1e-4 * np.abs(want) + 2e-6 * np.abs(want).max()
        bad = np.abs(got - want) > allow
        assert not bad.any(), "%s: %d of %d outside tolerance" % (what, bad.sum(), bad.size)

    close(g_w.cpu().numpy(), ref.G_W, "G_W")
    near = np.abs(np.abs(ref.G_Ht.astype(np.float64)) - 1.0) <= 2e-4
    close(np.where(~near, g_in.cpu().numpy(), 0), np.where(~near, ref.G_H, 0), "G_H")
    ctx.close()

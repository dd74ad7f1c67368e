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

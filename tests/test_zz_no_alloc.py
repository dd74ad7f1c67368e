"""The allocation-free layer entry point (collected last on purpose).

bigcn_layer_forward_noalloc() serves callers that cannot allocate device memory (a process whose
own pool already owns the whole GPU, or a loop that cannot take the stall of an allocation): its
scratch is a fixed array inside the library.  It must give what the layer of the paper gives (the
CPU oracle is the reference) and agree with bigcn_layer_forward(), call after call, although every
call reuses the same scratch and finds the previous call's leftovers in it.

The two CUDA entry points keep the integer dots in different storage between the contraction and
the aggregation (always 16-bit values here; bytes for some widths there), so their fp32 sums run in
different orders: H' and the next beta are compared within the tolerance, and a re-binarized bit may
differ only where the value under the sign sits at the threshold.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2210_13149_b200 import synth
from parity_util import ATOL, RTOL, bits_from_dev, bits_to_dev, dev, device_graph, flip_report, within_tol

pytestmark = pytest.mark.gpu


def _case(binding, n, e_dir, d_in, d_out, seed):
    """A layer problem and the oracle's results for it; the GPU side gets the oracle's packed input."""
    rng = np.random.default_rng(seed)
    rp, ci = synth.power_law_graph(n, e_dir, seed)
    src, dst = synth.edge_list(rp, ci)
    g = oracle.normalize_adjacency(n, src, dst)
    H = rng.standard_normal((n, d_in)).astype(np.float32)
    W = (rng.standard_normal((d_in, d_out)) * d_in ** -0.5).astype(np.float32)
    t = oracle.layer_forward(g, oracle.Layer(W), H)
    shift = (rng.standard_normal(d_out) * 0.01).astype(np.float32)
    scale = (rng.random(d_out) + 0.5).astype(np.float32)
    F_next, beta_next = oracle.binarize_rows(t.H_out, shift, scale)
    G = device_graph(binding, g)
    layer = binding.make_layer(d_in, d_out, bits_to_dev(t.bitsT), dev(t.alpha))
    dummy = torch.zeros((8, binding.packed_stride_words(d_out)), dtype=torch.int32).cuda()
    nxt = binding.make_layer(d_out, 8, dummy, torch.ones(8).cuda(), dev(shift), dev(scale))
    return dict(G=G, layer=layer, nxt=nxt, bits=bits_to_dev(t.bits), beta=dev(t.beta), H=t.H_out, shift=shift,
                F_next=F_next, beta_next=beta_next)


def test_noalloc_layer_matches_the_oracle_and_the_workspace_entry_point_twice_in_a_row():
    from paper_2210_13149_b200 import binding
    ctx = binding.BiGCN(0)
    # different problems, so that every call finds another one's leftovers in the scratch; the last one is large
    # enough (2^21 outputs, 4 MiB of scratch) for the contraction to run on the tensor cores
    cases = [_case(binding, 3000, 40000, 100, 256, 11), _case(binding, 5000, 30000, 602, 41, 12),
             _case(binding, 8192, 60000, 256, 256, 13)]
    refs = [ctx.layer_forward(c["G"], c["layer"], c["bits"], c["beta"], want_h=True, next_layer=c["nxt"]) for c in cases]
    ctx.sync_check()
    for round_ in range(2):
        for c, ref in zip(cases, refs):
            n, d_out = c["G"].n, c["layer"].d_out
            h = torch.full((n, d_out), float("nan"), device="cuda")
            nb = torch.full((n, binding.packed_stride_words(d_out)), -1, dtype=torch.int32, device="cuda")
            nbeta = torch.full((n,), float("nan"), device="cuda")
            st = binding.layer_forward_noalloc(c["G"], c["layer"], c["bits"], c["beta"], h, c["nxt"], nb, nbeta)
            assert st == 0
            torch.cuda.synchronize()
            ctx.sync_check()                                   # also reports a tensor-core wait that ran out
            # against the oracle
            ok, ratio, mx = within_tol(h, torch.from_numpy(c["H"]))
            assert ok, "H' against the oracle (round %d): error / allowance %.3g, max abs %.3g" % (round_, ratio, mx)
            flips, bad, total = flip_report(bits_from_dev(nb), c["F_next"], c["H"], c["shift"])
            assert bad == 0 and flips <= max(2, total // 2000), (flips, bad, total)
            np.testing.assert_allclose(nbeta.cpu().numpy(), c["beta_next"], rtol=RTOL, atol=ATOL)
            # against the entry point with a workspace
            ok, ratio, mx = within_tol(h, ref["h"])
            assert ok, "H' against bigcn_layer_forward (round %d): error / allowance %.3g" % (round_, ratio)
            differ = oracle.unpack_rows(bits_from_dev(nb), d_out) != oracle.unpack_rows(bits_from_dev(ref["next_bits"]), d_out)
            centred = c["H"].astype(np.float64) - c["shift"].astype(np.float64)[None, :]
            near = np.abs(centred) <= ATOL + RTOL * np.abs(c["H"].astype(np.float64))
            assert not (differ & ~near).any(), "re-binarized bits differ away from the threshold"
            np.testing.assert_allclose(nbeta.cpu().numpy(), ref["next_beta"].cpu().numpy(), rtol=RTOL, atol=ATOL)
            # pad bits of the packed rows are zero
            words = bits_from_dev(nb)
            if d_out % 32:
                assert (words[:, d_out // 32] >> (d_out % 32) == 0).all()
            assert (words[:, (d_out + 31) // 32:] == 0).all()
    ctx.close()


def test_noalloc_layer_refuses_what_does_not_fit():
    from paper_2210_13149_b200 import binding
    ctx = binding.BiGCN(0)
    d_in, d_out = 64, 256
    n = binding.NOALLOC_SCRATCH_BYTES // (d_out * 2) + 1       # one row too many for the built-in scratch
    rp, ci = synth.power_law_graph(n, 4 * n, 13, device="cuda")
    G = ctx.normalize_adjacency(rp, ci)
    gen = torch.Generator(device="cuda").manual_seed(13)
    bits, beta = ctx.pack_features(torch.randn((n, d_in), device="cuda", generator=gen))
    bitsT, alpha = ctx.pack_weights(torch.randn((d_in, d_out), device="cuda", generator=gen))
    layer = binding.make_layer(d_in, d_out, bitsT, alpha)
    h = torch.zeros((n, d_out), device="cuda")
    assert binding.layer_forward_noalloc(G, layer, bits, beta, h) == 5
    torch.cuda.synchronize()
    assert float(h.abs().sum()) == 0.0                         # nothing was launched
    # and bad arguments are refused without touching the GPU
    assert binding.layer_forward_noalloc(G, layer, bits, beta, None) == 1
    ctx.close()

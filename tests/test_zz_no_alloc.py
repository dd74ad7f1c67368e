"""The allocation-free layer entry point (collected last on purpose).

bigcn_layer_forward_noalloc() serves callers that cannot allocate device memory (a process whose
own pool already owns the whole GPU, or a loop that cannot take the stall of an allocation): its
scratch is a fixed array inside the library.  It must give what bigcn_layer_forward() gives, call
after call, although every call reuses the same scratch and finds the previous call's leftovers in it.
"""
import numpy as np
import pytest
import torch

from paper_2210_13149_b200 import synth

pytestmark = pytest.mark.gpu

ATOL, RTOL = 1e-4, 1e-5


def _case(binding, ctx, n, e_dir, d_in, d_out, seed):
    """A layer problem built with the library's own packers (existing entry points only)."""
    rp, ci = synth.power_law_graph(n, e_dir, seed, device="cuda")
    G = ctx.normalize_adjacency(rp, ci)
    g = torch.Generator(device="cuda").manual_seed(seed)
    H = torch.randn((n, d_in), device="cuda", generator=g)
    W = torch.randn((d_in, d_out), device="cuda", generator=g) * d_in ** -0.5
    W2 = torch.randn((d_out, 8), device="cuda", generator=g)
    bits, beta = ctx.pack_features(H)
    bitsT, alpha = ctx.pack_weights(W)
    layer = binding.make_layer(d_in, d_out, bitsT, alpha)
    b2, a2 = ctx.pack_weights(W2)
    shift = torch.randn(d_out, device="cuda", generator=g) * 0.01
    scale = torch.rand(d_out, device="cuda", generator=g) + 0.5
    nxt = binding.make_layer(d_out, 8, b2, a2, shift, scale)
    return G, layer, nxt, bits, beta


def _close(got, ref):
    return bool(((got.double() - ref.double()).abs() <= ATOL + RTOL * ref.double().abs()).all())


def test_noalloc_layer_matches_the_workspace_entry_point_twice_in_a_row():
    from paper_2210_13149_b200 import binding
    ctx = binding.BiGCN(0)
    # two different problems, so that the second call finds the first one's leftovers in the scratch
    cases = [_case(binding, ctx, 3000, 40000, 100, 256, 11), _case(binding, ctx, 5000, 30000, 602, 41, 12)]
    refs = []
    for G, layer, nxt, bits, beta in cases:
        refs.append(ctx.layer_forward(G, layer, bits, beta, want_h=True, next_layer=nxt))
    ctx.sync_check()
    for round_ in range(2):
        for (G, layer, nxt, bits, beta), ref in zip(cases, refs):
            n = G.n
            h = torch.full((n, layer.d_out), float("nan"), device="cuda")
            nb = torch.full((n, binding.packed_stride_words(layer.d_out)), -1, dtype=torch.int32, device="cuda")
            nbeta = torch.full((n,), float("nan"), device="cuda")
            st = binding.layer_forward_noalloc(G, layer, bits, beta, h, nxt, nb, nbeta)
            assert st == 0
            torch.cuda.synchronize()
            assert _close(h, ref["h"]), "H' differs (round %d)" % round_
            assert torch.equal(nb, ref["next_bits"])
            assert _close(nbeta, ref["next_beta"])
    ctx.close()


def test_noalloc_layer_refuses_what_does_not_fit():
    from paper_2210_13149_b200 import binding
    ctx = binding.BiGCN(0)
    d_out = 256
    n = binding.NOALLOC_SCRATCH_BYTES // (d_out * 2) + 1       # one row too many for the built-in scratch
    G, layer, nxt, bits, beta = _case(binding, ctx, n, 4 * n, 64, d_out, 13)
    h = torch.zeros((n, d_out), device="cuda")
    assert binding.layer_forward_noalloc(G, layer, bits, beta, h) == 5
    torch.cuda.synchronize()
    assert float(h.abs().sum()) == 0.0                         # nothing was launched
    # and bad arguments are refused without touching the GPU
    assert binding.layer_forward_noalloc(G, layer, bits, beta, None) == 1
    ctx.close()

"""bigcn_entropy_bins against the oracle's binning estimator (Sec. 6.2).

Range and interval counts are integer / comparison work decided in the same fp32 arithmetic on both
sides: exact.  Entropies are sums of p log2 p in double in a different order: relative 1e-12.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2210_13149_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2210_13149_b200 import binding
    c = binding.BiGCN(0)
    yield c
    c.close()


def activations(n, d, seed, kind="mixed"):
    """Synthetic hidden activations: per-neuron scale and offset, some neurons rectified, one constant,
    one two-valued (the shapes a trained layer shows; the trained values themselves are not available)."""
    rng = np.random.default_rng(seed)
    H = (rng.standard_normal((n, d)) * rng.uniform(0.2, 4.0, d) + rng.uniform(-1.0, 1.0, d)).astype(np.float32)
    if kind == "mixed" and d >= 4:
        H[:, 1] = np.maximum(H[:, 1], 0)
        H[:, 2] = 0.75
        H[:, 3] = np.where(rng.random(n) < 0.3, -2.0, 5.0)
    return H


def check(ctx, H, M):
    want = oracle.entropy_bins(H, M)
    got = ctx.entropy_bins(torch.from_numpy(H).cuda(), M)
    assert np.array_equal(got["col_min"].cpu().numpy(), want.col_min)
    assert np.array_equal(got["col_max"].cpu().numpy(), want.col_max)
    assert np.array_equal(got["counts"].cpu().numpy().astype(np.int64), want.counts)          # integers: exact
    np.testing.assert_allclose(got["entropy"].cpu().numpy(), want.entropy, rtol=1e-12, atol=1e-14)
    assert got["total"].item() == pytest.approx(want.total, rel=1e-12)
    return want


@pytest.mark.parametrize("n,d,M", [(1, 1, 1), (7, 3, 5), (1000, 16, 200), (4099, 33, 1000), (20011, 128, 1000),
                                   (3000, 50, 1024), (3000, 20, 1025), (2500, 9, 4096), (2500, 5, 8192), (100000, 7, 64)])
def test_entropy_bins_matches_oracle(ctx, n, d, M):
    check(ctx, activations(n, d, n * 31 + d), M)


def test_entropy_bins_strided_rows_and_repeat(ctx):
    rng = np.random.default_rng(3)
    buf = rng.standard_normal((5000, 40)).astype(np.float32)
    H = buf[:, :23]
    want = oracle.entropy_bins(np.ascontiguousarray(H), 300)
    dev = torch.from_numpy(buf).cuda()[:, :23]
    for _ in range(2):                                   # counts are overwritten, not accumulated
        got = ctx.entropy_bins(dev, 300)
        assert np.array_equal(got["counts"].cpu().numpy().astype(np.int64), want.counts)
        assert got["total"].item() == pytest.approx(want.total, rel=1e-12)


def test_entropy_bins_on_a_layer_output(ctx):
    """The estimator applied to what it is meant for: the fp32 output of a (binarized) layer."""
    from paper_2210_13149_b200 import binding as B
    wl = synth.make_workload("c3", device="cuda")
    G = ctx.normalize_adjacency(wl.rowptr.cuda(), wl.colidx.cuda())
    layers = ctx.prepare_layers([w.cuda() for w in wl.W])
    xb, xbeta = ctx.pack_features(wl.X.cuda())
    h = ctx.layer_forward(G, layers[0], xb, xbeta, want_h=True)["h"]
    want = check(ctx, h.cpu().numpy(), 200)
    assert 0 < want.total <= h.shape[1] * np.log2(200)


def test_entropy_bins_argument_checks(ctx):
    import ctypes
    H = torch.zeros((4, 4), device="cuda")
    out = ctx.entropy_bins(H, 3)                         # constant columns: everything in interval 0, zero entropy
    assert (out["counts"][:, 0] == 4).all() and (out["counts"][:, 1:] == 0).all() and out["total"].item() == 0.0
    from paper_2210_13149_b200 import binding as B
    with pytest.raises(B.BigcnError) as e:
        ctx.entropy_bins(H, 0)
    assert e.value.status == 2
    with pytest.raises(B.BigcnError) as e:
        ctx.entropy_bins(H, 8193)
    assert e.value.status == 7
    empty = ctx.entropy_bins(torch.zeros((0, 4), device="cuda"), 5)
    assert (empty["counts"] == 0).all() and (empty["entropy"] == 0).all() and empty["total"].item() == 0.0
    ctx.sync_check()

"""bigcn_pipeline_*: overlapped back-to-back forwards from host buffers.

Every submitted step must deliver exactly what bigcn_forward() delivers for the same input (the same
kernels run, only the copies overlap), in submission order, whatever the number of slots; the first
step is also held against the oracle.
"""
import numpy as np
import pytest
import torch

from paper_2210_13149_b200 import synth
from parity_util import ATOL, RTOL, dev, oracle_run

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2210_13149_b200 import binding
    return binding


@pytest.fixture(scope="module")
def net():
    return oracle_run(synth.make_workload("c3", device="cuda"), keep_trace=False)


def build(B, net):
    wl = net.wl
    ctx = B.BiGCN(0)
    G = ctx.normalize_adjacency(wl.rowptr.cuda(), wl.colidx.cuda())
    shifts = [dev(l.in_shift) if l.in_shift is not None else None for l in net.layers]
    scales = [dev(l.in_scale) if l.in_scale is not None else None for l in net.layers]
    layers = ctx.prepare_layers([w.cuda() for w in wl.W], shifts, scales)
    return ctx, G, layers


def step_inputs(wl, k):
    """Input of step k: the workload's features for k = 0, then seeded perturbations of them."""
    X = wl.X.cpu().clone()
    if k:
        g = torch.Generator().manual_seed(1000 + k)
        X = X + 0.5 * torch.randn(X.shape, generator=g)
    return X.contiguous()


@pytest.mark.parametrize("slots", [1, 2, 3, 5])
def test_pipeline_matches_forward_in_order(B, net, slots):
    ctx, G, layers = build(B, net)
    n_steps = 9
    xs = [step_inputs(net.wl, k).pin_memory() for k in range(n_steps)]
    want = [ctx.forward(G, layers, x.cuda()).cpu() for x in xs]
    outs = [torch.full((net.wl.n, want[0].shape[1]), float("nan")).pin_memory() for _ in range(n_steps)]
    pipe = ctx.open_pipeline(G, layers, slots=slots)
    done = 0
    for k in range(n_steps):
        if k - done == slots:                     # every slot is taken: drain the oldest step first
            got = pipe.wait()
            assert got is outs[done]
            assert torch.equal(got, want[done]), "step %d" % done
            done += 1
        pipe.submit(xs[k], outs[k])
    while done < n_steps:
        got = pipe.wait()
        assert torch.equal(got, want[done]), "step %d" % done
        done += 1
    assert pipe.wait() is None                    # nothing outstanding: returns at once
    pipe.close()
    # the first step is the workload itself: its predictions agree with the oracle's end-to-end run (what bigcn_forward
    # computes is held against the oracle element by element in test_gpu_parity.py and, below, for the packed steps)
    ref = torch.from_numpy(net.logits)
    assert (outs[0].argmax(1) == ref.argmax(1)).double().mean().item() > 0.99
    ctx.sync_check()
    ctx.close()


@pytest.mark.parametrize("slots", [1, 3])
def test_pipeline_steps_from_packed_input(B, net, slots):
    """Steps whose input is already binary (Sec. 5.2: packed sign bits and one scalar per node, in host memory), mixed
    with steps from fp32 features: bit for bit what bigcn_forward_packed() gives, and every logit within the tolerance of
    the oracle's last layer fed the very bits that layer saw (the network has two layers: the library's own
    re-binarized output of layer 0, unpacked by the oracle)."""
    import oracle
    from parity_util import bits_from_dev, within_tol
    ctx, G, layers = build(B, net)
    assert len(layers) == 2
    n_steps = 6
    xs = [step_inputs(net.wl, k) for k in range(n_steps)]
    packed = [ctx.pack_features(x.cuda(), layers[0].in_shift, layers[0].in_scale) for x in xs]
    want = [ctx.forward_packed(G, layers, b, be).cpu() for b, be in packed]
    for x, w in zip(xs, want):
        assert torch.equal(ctx.forward(G, layers, x.cuda()).cpu(), w)     # the same bits, the same result
    host = [(b.cpu().pin_memory(), be.cpu().pin_memory()) for b, be in packed]
    xs_pinned = [x.pin_memory() for x in xs]
    outs = [torch.full((net.wl.n, want[0].shape[1]), float("nan")).pin_memory() for _ in range(n_steps)]
    pipe = ctx.open_pipeline(G, layers, slots=slots)
    done = 0
    for k in range(n_steps):
        if k - done == slots:
            assert torch.equal(pipe.wait(), want[done]), "step %d" % done
            done += 1
        if k % 3 == 2:
            pipe.submit(xs_pinned[k], outs[k])                 # a step from fp32 features in between
        else:
            pipe.submit_packed(host[k][0], host[k][1], outs[k])
    while done < n_steps:
        assert torch.equal(pipe.wait(), want[done]), "step %d" % done
        done += 1
    pipe.close()
    # against the oracle, no element exempt
    for k in (0, 1):
        mid = ctx.layer_forward(G, layers[0], packed[k][0], packed[k][1], want_h=False, next_layer=layers[1])
        ref = oracle.layer_forward_packed(net.graph, net.layers[1], bits_from_dev(mid["next_bits"]), mid["next_beta"].cpu().numpy()).H_out
        ok, ratio, mx = within_tol(outs[k], torch.from_numpy(ref))
        assert ok, "step %d: error / allowance %.3g (max abs %.3g)" % (k, ratio, mx)
    ctx.sync_check()
    ctx.close()


def test_pipeline_refuses_more_steps_than_slots(B, net):
    ctx, G, layers = build(B, net)
    x = step_inputs(net.wl, 0).pin_memory()
    outs = [torch.empty((net.wl.n, layers[-1].d_out)).pin_memory() for _ in range(3)]
    pipe = ctx.open_pipeline(G, layers, slots=2)
    pipe.submit(x, outs[0])
    pipe.submit(x, outs[1])
    before = ctx.launch_count()
    with pytest.raises(B.BigcnError) as e:
        pipe.submit(x, outs[2])
    assert e.value.status == 9                    # BIGCN_ERR_BUSY
    assert ctx.launch_count() == before           # nothing was enqueued
    pipe.wait()
    pipe.submit(x, outs[2])                       # a slot is free again
    pipe.wait()
    pipe.wait()
    assert torch.equal(outs[0], outs[1]) and torch.equal(outs[0], outs[2])
    pipe.close()
    ctx.close()


def test_pipeline_argument_checks(B, net):
    import ctypes
    ctx, G, layers = build(B, net)
    arr = B._layer_array(layers)
    h = ctypes.c_void_p()
    ctx._prep_forward(G, layers, host_io=2)
    for bad_slots in (0, 9):
        st = ctx.lib.bigcn_pipeline_open(ctx.h, ctypes.byref(G.c), arr, len(layers), bad_slots, ctypes.byref(h))
        assert st == 2 and not h.value            # BIGCN_ERR_SHAPE
    # workspace sized for 2 slots, pipeline of 4: refused at submit, before anything is enqueued
    assert ctx.lib.bigcn_pipeline_open(ctx.h, ctypes.byref(G.c), arr, len(layers), 4, ctypes.byref(h)) == 0
    x = step_inputs(net.wl, 0).pin_memory()
    o = torch.empty((net.wl.n, layers[-1].d_out)).pin_memory()
    before = ctx.launch_count()
    st = ctx.lib.bigcn_pipeline_submit(h, ctypes.c_void_p(x.data_ptr()), ctypes.c_void_p(o.data_ptr()))
    assert st == 5                                # BIGCN_ERR_WORKSPACE
    assert ctx.lib.bigcn_pipeline_submit(h, None, ctypes.c_void_p(o.data_ptr())) in (1, 5)
    assert ctx.launch_count() == before
    assert ctx.lib.bigcn_pipeline_close(h) == 0
    ctx.sync_check()
    ctx.close()

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
    # the first step is the workload itself: hold it against the oracle
    ref = torch.from_numpy(net.logits)
    err = (outs[0].double() - ref.double()).abs()
    allow = ATOL + RTOL * ref.double().abs()
    assert (err > allow).double().mean().item() < 0.02      # threshold flips of re-binarised bits aside
    assert (outs[0].argmax(1) == ref.argmax(1)).double().mean().item() > 0.99
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

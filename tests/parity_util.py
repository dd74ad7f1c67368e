"""Shared helpers of the GPU parity tests: build a workload, run the CPU oracle on it, move arrays
to the device.  The oracle side and the CUDA side only meet here, through plain arrays."""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional

import numpy as np
import torch

import oracle
from paper_2210_13149_b200 import synth

ATOL, RTOL = 1e-4, 1e-5          # |gpu - oracle| <= ATOL + RTOL * |oracle| per fp32 element


def dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda()


def bits_to_dev(bits_u32: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits_u32).view(np.int32)).cuda()


def bits_from_dev(t: torch.Tensor) -> np.ndarray:
    return t.cpu().numpy().view(np.uint32)


def within_tol(got: torch.Tensor, ref: torch.Tensor):
    """Returns (ok, worst ratio of error to allowance, max abs error), computed where `got` lives."""
    ref = ref.to(got.device)
    err = (got.double() - ref.double()).abs()
    allow = ATOL + RTOL * ref.double().abs()
    ratio = (err / allow).max().item() if err.numel() else 0.0
    return ratio <= 1.0, ratio, (err.max().item() if err.numel() else 0.0)


def assert_close(got: torch.Tensor, ref, what=""):
    if isinstance(ref, np.ndarray):
        ref = torch.from_numpy(ref)
    assert got.shape == ref.shape, (what, got.shape, ref.shape)
    ok, ratio, mx = within_tol(got, ref)
    assert ok, "%s: error / allowance = %.3g (max abs err %.3g)" % (what, ratio, mx)


@dataclass
class OracleRun:
    wl: synth.Workload
    graph: oracle.Graph
    layers: List[oracle.Layer]
    traces: Optional[List[oracle.LayerTrace]]
    logits: np.ndarray


def oracle_run(wl: synth.Workload, keep_trace=True) -> OracleRun:
    src, dst = synth.edge_list(wl.rowptr, wl.colidx)
    g = oracle.normalize_adjacency(wl.n, src, dst)
    X = wl.X.cpu().numpy()
    W = [w.cpu().numpy() for w in wl.W]
    layers = oracle.calibrate_bn(g, W, X, wl.bn_layers())
    logits, traces = oracle.forward(g, layers, X, keep_trace=keep_trace)
    return OracleRun(wl, g, layers, traces if keep_trace else None, logits)


def device_graph(binding, g: oracle.Graph):
    return binding.make_graph(dev(g.rowptr), dev(g.colidx), dev(g.val), dev(g.dinv))


def device_layers_from_oracle(binding, run: OracleRun):
    """Layers whose packed weights, alpha and batch-norm constants are the oracle's own arrays."""
    out = []
    for l, layer in enumerate(run.layers):
        B, alpha = oracle.binarize_cols(layer.W)
        bitsT = oracle.pack_cols(B)
        sh = dev(layer.in_shift) if layer.in_shift is not None else None
        sc = dev(layer.in_scale) if layer.in_scale is not None else None
        out.append(binding.make_layer(layer.W.shape[0], layer.W.shape[1], bits_to_dev(bitsT), dev(alpha), sh, sc))
    return out


def flip_report(gpu_bits: np.ndarray, ref_F: np.ndarray, ref_H: np.ndarray, shift: Optional[np.ndarray]):
    """Compares re-binarized bits with the oracle's signs.  A disagreement is admissible only where
    the oracle's pre-sign value lies within the fp32 tolerance of the threshold.
    Returns (flips, inadmissible flips, total)."""
    d = ref_F.shape[1]
    got_F = oracle.unpack_rows(gpu_bits, d)
    diff = got_F != ref_F
    centred = ref_H.astype(np.float64) - (shift.astype(np.float64)[None, :] if shift is not None else 0.0)
    near = np.abs(centred) <= ATOL + RTOL * np.abs(ref_H.astype(np.float64))
    bad = diff & ~near
    return int(diff.sum()), int(bad.sum()), int(diff.size)


def unpack_signs_dev(bits: torch.Tensor, d: int) -> torch.Tensor:
    """bool [n, d] from packed int32 words [n, stride] (bit k of word w is element 32 w + k)."""
    n = bits.shape[0]
    shifts = torch.arange(32, device=bits.device, dtype=torch.int32)
    b = (bits.unsqueeze(-1) >> shifts) & 1
    return b.reshape(n, -1)[:, :d].bool()


def end_to_end_with_flip_accounting(ctx, G, layers, run: OracleRun, X: torch.Tensor):
    """Runs the network layer by layer on the GPU's own intermediate results and checks EVERY row of
    EVERY layer against the oracle -- no row is exempt:

    * layer 0 gets the same packed input on both sides (asserted bit for bit), so its output is
      compared with the oracle's own layer 0;
    * every later layer is compared with the oracle's layer fed the GPU's own packed input (the
      re-binarized bits unpacked by the oracle, and the GPU's beta): all rows of H' within the
      tolerance, re-binarized bits equal to the sign of that reference except where the reference
      lies within the tolerance of the threshold, the next beta within the tolerance -- for the launch
      that also writes H' and for the launch that wants only bits and beta (what bigcn_forward runs
      for a hidden layer; its outputs feed the next layer here as they do there).

    Beside that it keeps the accounting against the oracle's own end-to-end run (whose later layers
    see the oracle's bits, so a threshold flip moves the rows downstream of it): threshold flips per
    layer, share of logit rows downstream of a flip, share of logits outside tolerance, argmax
    agreement.  Those figures are reported, not asserted, except that a flip which is not itself
    downstream of an earlier one must sit at the threshold."""
    n = G.n
    A = torch.sparse_csr_tensor(G.rowptr, G.colidx.long(), torch.ones_like(G.val), size=(n, n))
    L = len(layers)
    bits, beta = ctx.pack_features(X, layers[0].in_shift, layers[0].in_scale)
    assert torch.equal(bits, bits_to_dev(run.traces[0].bits)), "first-layer packed bits differ from the oracle"
    dirty = torch.zeros(n, dtype=torch.bool, device=X.device)          # rows whose packed input differs
    report = {"origin_flips": [], "dirty_rows": [], "own_fed_flips": [], "own_fed_worst_ratio": []}
    for l in range(L):
        t = run.traces[l]
        nxt = layers[l + 1] if l + 1 < L else None
        out = ctx.layer_forward(G, layers[l], bits, beta, want_h=True, next_layer=nxt)
        # ---- the complete check: the oracle's layer on the very input the GPU's layer saw
        if l == 0:
            own_H = t.H_out
        else:
            own_H = oracle.layer_forward_packed(run.graph, run.layers[l], bits_from_dev(bits), beta.cpu().numpy()).H_out
        ok, ratio, mx = within_tol(out["h"], torch.from_numpy(own_H))
        assert ok, "layer %d on the GPU's own input: H' error / allowance = %.3g (max abs %.3g)" % (l, ratio, mx)
        report["own_fed_worst_ratio"].append(ratio)
        if nxt is not None:
            nl = run.layers[l + 1]
            own_F, own_beta = oracle.binarize_rows(own_H, nl.in_shift, nl.in_scale)
            flips, bad, total = flip_report(bits_from_dev(out["next_bits"]), own_F, own_H, nl.in_shift)
            assert bad == 0, "layer %d on the GPU's own input: %d of %d sign flips away from the threshold" % (l, bad, flips)
            np.testing.assert_allclose(out["next_beta"].cpu().numpy(), own_beta, rtol=RTOL, atol=ATOL)
            # the same layer as bigcn_forward launches it -- only the sign bits and beta wanted, which may run another
            # aggregation kernel -- held to the same reference; its outputs are the ones carried to the next layer
            carried = ctx.layer_forward(G, layers[l], bits, beta, want_h=False, next_layer=nxt)
            flips, bad, total = flip_report(bits_from_dev(carried["next_bits"]), own_F, own_H, nl.in_shift)
            assert bad == 0, "layer %d (bits only) on the GPU's own input: %d of %d sign flips away from the threshold" % (l, bad, flips)
            report["own_fed_flips"].append(flips)
            np.testing.assert_allclose(carried["next_beta"].cpu().numpy(), own_beta, rtol=RTOL, atol=ATOL)
            out["next_bits"], out["next_beta"] = carried["next_bits"], carried["next_beta"]
            del own_F, own_beta, carried
        del own_H
        # ---- accounting against the oracle's own end-to-end run
        tainted = (A @ dirty.to(torch.float32).unsqueeze(1)).squeeze(1) > 0    # rows that gather a differing row
        ref = dev(t.H_out)
        err = (out["h"].double() - ref.double()).abs()
        allow = ATOL + RTOL * ref.double().abs()
        clean_bad = ((err > allow).any(1) & ~tainted).sum().item()
        assert clean_bad == 0, "layer %d: %d rows outside tolerance that no sign flip explains" % (l, clean_bad)
        if nxt is None:
            report["logit_rows_downstream_of_flips"] = float(tainted.double().mean())
            report["logits_outside_tolerance"] = float((err > allow).double().mean())
            report["max_abs_err"] = float(err.max())
            report["argmax_agreement"] = float((out["h"].argmax(1) == ref.argmax(1)).double().mean())
            break
        tn = run.traces[l + 1]
        got = unpack_signs_dev(out["next_bits"], layers[l].d_out)
        want = dev(tn.F) > 0
        diff = got != want
        mu = dev(run.layers[l + 1].in_shift).double() if run.layers[l + 1].in_shift is not None else 0.0
        near = (ref.double() - mu).abs() <= allow
        origin = diff & ~tainted.unsqueeze(1)
        bad = int((origin & ~near).sum())
        assert bad == 0, "layer %d: %d sign flips away from the threshold" % (l, bad)
        report["origin_flips"].append(int(origin.sum()))
        dirty = diff.any(1) | (err > allow).any(1)       # rows whose packed bits or scale are no longer the oracle's
        report["dirty_rows"].append(int(dirty.sum()))
        bits, beta = out["next_bits"], out["next_beta"]
        del out, got, want, diff, near, origin, err, allow, ref
    return report

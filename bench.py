#!/usr/bin/env python
"""Benchmark of the Bi-GCN binarized forward path: nodes/s of a full L-layer forward on one B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config c5] [--impl ours|reference]

A step is one pass of the whole hot path (binarize+pack of the fp32 features, then per layer the
XNOR/bit-count contraction with rescale and the CSR aggregation with fused re-binarization) over one
seeded synthetic graph.  With N > 1 every rank runs an independent replica on its own GPU (the path
has no exchange step); the reported value is the sum over replicas divided by the slowest rank's time.
Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "bigcn_forward_nodes_per_s"
UNIT = "nodes/s"
DTYPE = "u32-xor-popc+f32"                # contraction on the XOR / bit-count pipe, fp32 aggregation
DTYPE_TC = "b1-as-s8-tcgen05-s32+f32"     # contraction as int8 tensor-core products of the +-1 bits (int32 sums), fp32 aggregation


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", default="c5", help="workload c1..c5 (default: the largest, c5)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--model", default="gcn", choices=["gcn", "sage", "entropy", "backward"],
                    help="gcn: the Bi-GCN forward (the benchmark); sage: side benchmark of the Bi-GraphSAGE layers; "
                         "entropy: side benchmark of the binning entropy estimator; backward: side benchmark of Algorithm 1 "
                         "for the hidden layer of the workload")
    ap.add_argument("--zeta-format", type=int, default=0, help="0 auto, 1 fp32, 2 int16, 3 int8, 4 fp16, 5 half-dot bytes")
    ap.add_argument("--byte-aggregation", type=int, default=0,
                    help="rows of 129..256 bytes: 0 the library's choice (tcgen05 products for hidden layers), 1 the fp32 FMA stream, "
                         "2 integer products on mma.sync, 3 tcgen05 products wherever they apply")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--graph", action="store_true", help="also time the forward replayed as one CUDA graph")
    ap.add_argument("--cpu-sample-scale", type=float, default=None)
    ap.add_argument("--scale", type=float, default=None,
                    help="shrink nodes and edges of the workload by this factor (profiling on a small case)")
    return ap.parse_args()


def workload_description(spec, n, nnz):
    return ("%s: %d-layer Bi-GCN forward, synthetic power-law graph, %d nodes, %d stored entries of A_tilde, "
            "widths %s, %s features" % (spec.name, len(spec.dims) - 1, n, nnz, "-".join(str(d) for d in spec.dims),
                                        spec.features))


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            with open(path) as f:
                p = json.load(f)
            return float(p["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.out = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.FIELDS,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=self.out, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.out.close()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            for line in open(self.path):
                parts = [p.strip() for p in line.split(",")]
                if len(parts) < 9:
                    continue
                try:
                    sm.append(float(parts[1]))
                    mx.append(float(parts[2]))
                except ValueError:
                    continue
                for name, v in zip(names, parts[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------------------------- oracle arm

def time_oracle(spec_name: str, scale: float, steps: int, warmup: int):
    """Times the CPU oracle, as it stands, on the workload itself (scale 1) or on a scaled-down draw of it (same
    recipe, same widths and mean degree).  The inputs are drawn on the GPU when there is one (the large graphs take
    minutes to draw on a CPU) and handed to the oracle as host arrays; every timed step is a full oracle forward on
    the host cores.  Returns (nodes/s, threads, sample description, ms per step, nodes, stored entries)."""
    import torch
    import oracle
    from paper_2210_13149_b200 import synth
    draw_on = "cuda" if torch.cuda.is_available() else "cpu"
    wl = synth.make_workload(spec_name, scale=scale if scale < 1.0 else None, device=draw_on)
    src, dst = synth.edge_list(wl.rowptr, wl.colidx)
    g = oracle.normalize_adjacency(wl.n, src, dst)
    X = wl.X.cpu().numpy()
    W = [w.cpu().numpy() for w in wl.W]
    n = wl.n
    bn = wl.bn_layers()
    del wl, src, dst
    if draw_on == "cuda":
        torch.cuda.empty_cache()
    layers = oracle.calibrate_bn(g, W, X, bn)
    times = []
    for it in range(warmup + steps):
        t0 = time.perf_counter()
        oracle.forward(g, layers, X, keep_trace=False)
        t1 = time.perf_counter()
        if it >= warmup:
            times.append(t1 - t0)
    ms = 1e3 * sum(times) / len(times)
    if scale < 1.0:
        sample = ("%s recipe at %g of its nodes and edges (%d nodes, %d stored entries, same widths and mean degree): "
                  "full %d-layer oracle forward, set-up excluded" % (spec_name, scale, n, g.nnz, len(layers)))
    else:
        sample = ("the whole workload %s (%d nodes, %d stored entries): full %d-layer oracle forward, set-up excluded, "
                  "%d timed steps after %d warm-up" % (spec_name, n, g.nnz, len(layers), steps, warmup))
    return n / (ms * 1e-3), oracle.num_threads(), sample, ms, n, g.nnz


def oracle_work(spec) -> float:
    """Multiply-adds of one oracle forward: the aggregation's nnz x d_out per layer plus the bit-count contraction."""
    return sum(spec.e_dir * d for d in spec.dims[1:]) + sum(spec.n * a * b / 32 for a, b in zip(spec.dims[:-1], spec.dims[1:]))


def default_cpu_scale(spec, forwards: int = 5, budget_s: float = 150.0) -> float:
    """The oracle runs on the workload itself when `forwards` forwards (warm-up, timed steps and the one that freezes
    the batch-norm constants) fit the time budget on this host -- about 1e9 multiply-adds per second and core, as
    measured -- and on a scaled-down draw otherwise."""
    cores = max(1, os.cpu_count() or 1)
    seconds_full = oracle_work(spec) / (0.9e9 * min(cores, 32)) * forwards
    return 1.0 if seconds_full <= budget_s else max(0.01, budget_s / seconds_full)


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2210_13149_b200 import synth
    spec = synth.WORKLOADS[args.config]
    scale = args.cpu_sample_scale or default_cpu_scale(spec, forwards=args.steps + args.warmup + 1)
    value, threads, sample, ms, n, nnz = time_oracle(args.config, scale, args.steps, args.warmup)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64-accumulate (CPU oracle)", "data": "synthetic",
            "config": {"workload": workload_description(spec, n, nnz) if scale >= 1.0 else
                       workload_description(spec, spec.n, spec.e_dir + spec.n) + " (the CPU oracle, timed on a sample of it)",
                       "l2": "inputs_exceed_l2", "parallelism": "single-gpu", "zeta_format": "auto", "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------------------------- our arm

L2_BYTES = 126e6


def spmm_bytes_model(n, nnz, row_bytes, out_bytes, deg_desc_cumsum=None):
    """Algorithmic HBM bytes of one aggregation launch.

    Fixed part: the CSR stream (4-byte column + 4-byte value per stored entry), rowptr, the
    per-node weight vector and the output.  Operand rows: `lower` reads every row once (perfect
    reuse), `upper` reads one row per stored entry (no reuse).  `cached` is the figure used for the
    roofline: every row once, plus one row per stored entry whose source node is not among the
    rows an ideal 126 MB cache would keep resident, i.e. the highest-degree nodes (a node is
    gathered once per incident entry, and node ids carry no other locality)."""
    fixed = nnz * 8.0 + 8.0 * (n + 1) + 4.0 * n + out_bytes
    z = n * row_bytes
    lower = fixed + z
    upper = fixed + nnz * row_bytes
    cached = upper
    if deg_desc_cumsum is not None and n > 0:
        k = int(min(n, L2_BYTES // row_bytes))                 # rows the ideal cache holds
        hit_entries = float(deg_desc_cumsum[k - 1]) - k if k > 0 else 0.0   # their gathers after the first
        cached = fixed + z + max(0.0, (nnz - n) - hit_entries) * row_bytes
    return lower, upper, cached


def traffic_record(kernel_key):
    """DRAM bytes per launch of the dominant kernel from the committed ncu capture, or None when
    the kernel source has changed since the counters were taken."""
    import hashlib
    path = os.path.join(ROOT, "profiles", "traffic_records.json")
    try:
        rec = json.load(open(path))[kernel_key]
        src = os.path.join(ROOT, "paper_2210_13149_b200", "csrc", rec["source"])
        if hashlib.sha256(open(src, "rb").read()).hexdigest() != rec["source_sha256"]:
            return None
        return float(rec["dram_bytes_per_launch"])
    except Exception:
        return None


def run_ours(args):
    import torch
    from paper_2210_13149_b200 import binding, replicas, synth

    rank, local, world = replicas.env_rank()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    replicas.init("nccl", dev)

    wl = synth.make_workload(args.config, scale=args.scale, device=dev)
    spec = wl.spec
    ctx = binding.BiGCN(local)
    if args.zeta_format:
        ctx.set_option(binding.OPT_ZETA_FORMAT, args.zeta_format)
    if args.byte_aggregation:
        ctx.set_option(binding.OPT_BYTE_AGGREGATION, args.byte_aggregation)
    G = ctx.normalize_adjacency(wl.rowptr, wl.colidx)
    n, nnz = G.n, G.nnz
    deg = torch.sort(torch.diff(G.rowptr), descending=True).values
    deg_cum = torch.cumsum(deg, 0).cpu().numpy()               # for the cache-aware byte model of the aggregation
    del deg
    del wl.rowptr, wl.colidx
    dims = list(spec.dims)
    L = len(dims) - 1

    # Set-up (untimed): pack the weights; freeze the batch-norm constants of every layer input that
    # has them from the library's own column statistics, layer after layer.
    bn = wl.bn_layers()
    packed = [ctx.pack_weights(W) for W in wl.W]
    layers, shifts, scales = [], [], []
    bits = beta = None
    for l in range(L):
        if l == 0:
            sh, sc = ctx.col_stats(wl.X) if bn[0] else (None, None)
            bits, beta = ctx.pack_features(wl.X, sh, sc)
        else:
            prev = layers[-1]
            out = ctx.layer_forward(G, prev, bits, beta, want_h=True)
            sh, sc = ctx.col_stats(out["h"]) if bn[l] else (None, None)
            bits, beta = ctx.pack_features(out["h"], sh, sc)
            del out
        layers.append(binding.make_layer(dims[l], dims[l + 1], packed[l][0], packed[l][1], sh, sc))
    del bits, beta
    ctx.workspace = None
    torch.cuda.empty_cache()

    X = wl.X
    logits = torch.empty((n, dims[-1]), dtype=torch.float32, device=dev)
    ctx._prep_forward(G, layers, host_io=not args.no_e2e)

    def barrier():
        replicas.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        ctx.forward(G, layers, X, logits)
    barrier()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    launches0 = ctx.launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    per_kernel = {"pack": [], "gemm": [[] for _ in range(L)], "spmm": [[] for _ in range(L)], "step": []}
    barrier()
    ev0.record()
    for _ in range(args.steps):
        _, st = ctx.forward(G, layers, X, logits, stats=True)
        per_kernel["pack"].append(st.ms_pack)
        per_kernel["step"].append(st.ms_total)
        for l in range(L):
            per_kernel["gemm"][l].append(st.ms_gemm[l])
            per_kernel["spmm"][l].append(st.ms_spmm[l])
    ev1.record()
    barrier()
    elapsed_ms = ev0.elapsed_time(ev1)
    launches = ctx.launch_count() - launches0
    clocks = sampler.stop() if rank == 0 else None
    value, ms_per_step = replicas.throughput(elapsed_ms / args.steps, n, dev)

    # side measurements (not part of `value`): the same forward from already-binary input (Sec. 5.2 of
    # the paper: the loaded data is binary), and replayed as one CUDA graph (the small workloads are
    # bound by launch latency)
    extras = {}
    if rank == 0:
        xb, xbeta = ctx.pack_features(X, layers[0].in_shift, layers[0].in_scale)
        for _ in range(3):
            ctx.forward_packed(G, layers, xb, xbeta, logits)
        barrier_local = torch.cuda.synchronize
        barrier_local()
        ev0.record()
        for _ in range(args.steps):
            ctx.forward_packed(G, layers, xb, xbeta, logits)
        ev1.record()
        barrier_local()
        extras["packed_input_ms_per_step"] = ev0.elapsed_time(ev1) / args.steps
        del xb, xbeta
        if args.graph or ms_per_step < 2.0:
            try:
                side = torch.cuda.Stream()
                gctx = binding.BiGCN(local, stream=side)
                gctx._prep_forward(G, layers)
                with torch.cuda.stream(side):
                    for _ in range(3):
                        gctx.forward(G, layers, X, logits)
                side.synchronize()
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph, stream=side):
                    gctx.forward(G, layers, X, logits)
                for _ in range(3):
                    graph.replay()
                torch.cuda.synchronize()
                reps = max(args.steps, 50)
                ev0.record()
                for _ in range(reps):
                    graph.replay()
                ev1.record()
                torch.cuda.synchronize()
                extras["cuda_graph_ms_per_step"] = ev0.elapsed_time(ev1) / reps
                del graph
                gctx.close()
            except Exception as exc:
                extras["cuda_graph_ms_per_step"] = "failed: %r" % (exc,)
        try:
            extras["popc_word_steps_per_s"] = ctx.measure_popc_peak()
        except Exception as exc:
            extras["popc_word_steps_per_s"] = None
        # the same forward with every zeta row in fp16 (the HBM-bound variant of the wide aggregations), for comparison
        if args.zeta_format == 0:
            try:
                ctx.set_option(binding.OPT_ZETA_FORMAT, binding.ZETA_F16)
                alt = [[] for _ in range(L)]
                for k in range(3 + min(args.steps, 5)):
                    _, st = ctx.forward(G, layers, X, logits, stats=True)
                    if k >= 3:
                        for l in range(L):
                            alt[l].append(st.ms_spmm[l])
                extras["spmm_fp16_rows_ms"] = [sum(v) / len(v) for v in alt]
            except Exception as exc:
                extras["spmm_fp16_rows_ms"] = "failed: %r" % (exc,)
            finally:
                ctx.set_option(binding.OPT_ZETA_FORMAT, 0)
        # byte rows aggregated by the library's other paths, for comparison: the fp32 FMA stream (1) and integer
        # products on mma.sync (2); the default for a hidden layer of 129..256 byte columns is tcgen05 products (3)
        if args.zeta_format == 0 and args.byte_aggregation == 0:
            for opt, key in ((1, "spmm_fma_stream_ms"), (2, "spmm_integer_products_ms")):
                try:
                    ctx.set_option(binding.OPT_BYTE_AGGREGATION, opt)
                    alt = [[] for _ in range(L)]
                    for k in range(3 + min(args.steps, 5)):
                        _, st = ctx.forward(G, layers, X, logits, stats=True)
                        if k >= 3:
                            for l in range(L):
                                alt[l].append(st.ms_spmm[l])
                    extras[key] = [sum(v) / len(v) for v in alt]
                except Exception as exc:
                    extras[key] = "failed: %r" % (exc,)
                finally:
                    ctx.set_option(binding.OPT_BYTE_AGGREGATION, 0)
        # the gather of the aggregations alone (no weights, no sums, no output): what the memory system needs for the
        # row sizes this network's layers store
        try:
            extras["gather_only_ms"] = {str(rb): ctx.measure_gather_peak(G, rb) for rb in (256, 64)}
        except Exception as exc:
            extras["gather_only_ms"] = "failed: %r" % (exc,)
        # the same contraction on the XOR / bit-count pipe (the library's other path), for comparison
        try:
            ctx.set_option(binding.OPT_CONTRACTION, 1)
            pop = [[] for _ in range(L)]
            for k in range(3 + min(args.steps, 5)):
                _, st = ctx.forward(G, layers, X, logits, stats=True)
                if k >= 3:
                    for l in range(L):
                        pop[l].append(st.ms_gemm[l])
            extras["bitgemm_popc_pipe_ms"] = [sum(v) / len(v) for v in pop]
        except Exception as exc:
            extras["bitgemm_popc_pipe_ms"] = "failed: %r" % (exc,)
        finally:
            ctx.set_option(binding.OPT_CONTRACTION, 0)

    # end to end through the host-buffer entry points: every step copies its input from pinned host
    # memory and its logits back to pinned host memory.  Headline: the pipelined entry point (the
    # upload of step k+1 and the download of step k-1 overlap the forward of step k); the one-step-at-
    # a-time call is timed beside it.
    e2e = None
    if not args.no_e2e:
        slots = 3
        xh = [torch.empty((n, dims[0]), dtype=torch.float32).pin_memory() for _ in range(slots)]
        for t in xh:
            t.copy_(X)
        oh = [torch.empty((n, dims[-1]), dtype=torch.float32).pin_memory() for _ in range(slots)]
        e_steps = max(3, min(args.steps, 10))
        for _ in range(2):
            ctx.forward_host(G, layers, xh[0], oh[0])
        barrier()
        ev0.record()
        for _ in range(e_steps):
            ctx.forward_host(G, layers, xh[0], oh[0])
        ev1.record()
        barrier()
        sync_value, sync_ms = replicas.throughput(ev0.elapsed_time(ev1) / e_steps, n, dev)

        pipe = ctx.open_pipeline(G, layers, slots=slots)

        def run_pipelined(k_steps):
            outstanding = 0
            for k in range(k_steps):
                if outstanding == slots:
                    pipe.wait()
                    outstanding -= 1
                pipe.submit(xh[k % slots], oh[k % slots])
                outstanding += 1
            while outstanding:
                pipe.wait()
                outstanding -= 1

        run_pipelined(slots)                      # warm-up: every slot used once
        p_steps = max(2 * e_steps, 4 * slots)         # long enough that filling and draining the pipeline is a small share
        barrier()
        t0 = time.perf_counter()
        ev0.record()
        run_pipelined(p_steps)                    # returns when the last logits are in host memory
        ev1.record()
        wall_ms = (time.perf_counter() - t0) * 1e3
        barrier()
        # the device events bracket the compute stream only; the copies of the last steps end later, so
        # the host clock around the whole loop (which ends with the last delivery) is the honest one
        e_value, e_ms = replicas.throughput(max(wall_ms, ev0.elapsed_time(ev1)) / p_steps, n, dev)

        # the same pipeline fed an input that is already binary (Sec. 5.2: 1 bit per element + one scalar per node)
        xb_dev, xbeta_dev = ctx.pack_features(X, layers[0].in_shift, layers[0].in_scale)
        bh = [xb_dev.cpu().pin_memory() for _ in range(slots)]
        beh = [xbeta_dev.cpu().pin_memory() for _ in range(slots)]
        packed_in_bytes = xb_dev.numel() * 4 + xbeta_dev.numel() * 4
        del xb_dev, xbeta_dev

        def run_pipelined_packed(k_steps):
            outstanding = 0
            for k in range(k_steps):
                if outstanding == slots:
                    pipe.wait()
                    outstanding -= 1
                pipe.submit_packed(bh[k % slots], beh[k % slots], oh[k % slots])
                outstanding += 1
            while outstanding:
                pipe.wait()
                outstanding -= 1

        run_pipelined_packed(slots)
        barrier()
        t0 = time.perf_counter()
        ev0.record()
        run_pipelined_packed(p_steps)
        ev1.record()
        wall_packed_ms = (time.perf_counter() - t0) * 1e3
        barrier()
        pipe.close()
        pk_value, pk_ms = replicas.throughput(max(wall_packed_ms, ev0.elapsed_time(ev1)) / p_steps, n, dev)
        del bh, beh
        e2e = {"value": e_value, "unit": UNIT, "ms_per_step": e_ms, "steps": p_steps,
               "h2d_bytes_per_step": n * dims[0] * 4, "d2h_bytes_per_step": n * dims[-1] * 4,
               "api": "bigcn_pipeline_submit/wait, %d slots (pinned host X in, host logits out, every step; "
                      "copies of neighbouring steps overlap the forward)" % slots,
               "one_step_at_a_time": {"value": sync_value, "ms_per_step": sync_ms, "steps": e_steps,
                                      "api": "bigcn_forward_host"},
               "packed_input": {"value": pk_value, "unit": UNIT, "ms_per_step": pk_ms, "steps": p_steps,
                                "h2d_bytes_per_step": packed_in_bytes, "d2h_bytes_per_step": n * dims[-1] * 4,
                                "api": "bigcn_pipeline_submit_packed/wait, %d slots (pinned host sign bits + beta in, host "
                                       "logits out, every step)" % slots}}
        del xh, oh

    if rank != 0:
        replicas.finish()
        return

    # roofline of the dominant kernel: the aggregation of the layer that takes longest
    peak, peak_kind = load_peaks()
    mean = lambda v: sum(v) / len(v)
    spmm_ms = [mean(v) for v in per_kernel["spmm"]]
    gemm_ms = [mean(v) for v in per_kernel["gemm"]]
    pack_ms = mean(per_kernel["pack"])
    kernels = {}
    dom = max(range(L), key=lambda l: spmm_ms[l])
    for l in range(L):
        f = args.zeta_format                      # the library's rule for the storage of zeta, layer by layer
        wide = 128 < dims[l + 1] <= 256 or (l == L - 1 and 32 < dims[l + 1] <= 64)   # (a last layer: fp32 output only)
        half_ok = dims[l + 1] <= 256 and 128 <= dims[l] <= 256 and n >= 64
        if f == 0:
            if wide and dims[l] <= 127:
                f = binding.ZETA_I8
            elif half_ok and wide and n * dims[l + 1] >= (1 << 20):
                f = binding.ZETA_I8H
            else:
                f = binding.ZETA_F16
        if f == binding.ZETA_I8H and not half_ok:
            f = binding.ZETA_I8 if (wide and dims[l] <= 127) else binding.ZETA_F16
        if f == binding.ZETA_I8 and dims[l] > 127:
            f = binding.ZETA_F16
        if f == binding.ZETA_F16 and dims[l] > 2048:
            f = binding.ZETA_I16
        elt = {1: 4, 2: 2, 3: 1, 4: 2, 5: 1}[f]
        per16 = 16 // elt
        ldz = (dims[l + 1] + per16 - 1) // per16 * per16
        last = (l == L - 1)
        # a last layer of 33..60 byte columns on the tensor-core contraction: 64-byte rows that carry the node factor
        on_tc = dims[l] <= 256 and dims[l + 1] <= 256 and (f == binding.ZETA_I8H or n * dims[l + 1] >= (1 << 20))
        if last and elt == 1 and 32 < dims[l + 1] <= 60 and on_tc:
            ldz = 64
        out_bytes = n * dims[l + 1] * 4.0 if last else n * (binding.packed_stride_words(dims[l + 1]) * 4.0 + 4.0)
        lower, upper, expected = spmm_bytes_model(n, nnz, ldz * elt, out_bytes, deg_cum)
        t = spmm_ms[l] * 1e-3
        # the library's rule for the aggregation kernel: tcgen05 products for a hidden layer (only bits and beta wanted) of
        # 129..256 byte columns on a graph whose rows average at least 8 stored entries, unless another path is asked for
        on_tc_agg = (elt == 1 and 128 < dims[l + 1] <= 256 and not last and nnz < (1 << 31)
                     and (args.byte_aggregation == 3 or (args.byte_aggregation == 0 and nnz >= 8 * n)))
        agg_name = "spmm_tc_kernel" if on_tc_agg else ("spmm_lane_kernel" if (last and elt == 1 and 32 < dims[l + 1] <= 64 and nnz >= 8 * n) else "spmm_kernel")
        kernels["spmm_l%d" % l] = {"ms": spmm_ms[l], "kernel": agg_name, "GBps_cached_model": expected / t / 1e9,
                                   "GBps_lower_model": lower / t / 1e9, "GBps_no_reuse_model": upper / t / 1e9,
                                   "bytes_cached_model": expected, "row_bytes": ldz * elt, "zeta_format": {1: "f32", 2: "i16", 3: "i8", 4: "f16", 5: "i8h"}[f]}
        ops = 2.0 * n * dims[l] * dims[l + 1]
        words = n * dims[l + 1] * ((dims[l] + 31) // 32)                  # XOR + bit-count + add steps
        popc_peak = extras.get("popc_word_steps_per_s")
        on_tc = dims[l] <= 256 and dims[l + 1] <= 256 and (n * dims[l + 1] >= (1 << 20) or f == binding.ZETA_I8H)   # the library's rule for the tensor-core path
        k_pad = binding.packed_stride_words(dims[l]) * 32
        io_bytes = n * (binding.packed_stride_words(dims[l]) * 4.0 + 4.0 + ldz * elt)
        kernels["bitgemm_l%d" % l] = {"ms": gemm_ms[l], "path": "tcgen05 int8" if on_tc else "xor+popc",
                                      "binary_TOPS": ops / (gemm_ms[l] * 1e-3) / 1e12,
                                      "int8_TOPS_issued": (2.0 * n * k_pad * dims[l + 1] / (gemm_ms[l] * 1e-3) / 1e12) if on_tc else None,
                                      "word_steps_per_s": words / (gemm_ms[l] * 1e-3),
                                      "frac_of_popc_peak": (words / (gemm_ms[l] * 1e-3) / popc_peak) if popc_peak else None,
                                      "out_GBps": n * ldz * elt / (gemm_ms[l] * 1e-3) / 1e9,
                                      "GBps": io_bytes / (gemm_ms[l] * 1e-3) / 1e9,
                                      "frac_of_hbm_peak": io_bytes / (gemm_ms[l] * 1e-3) / 1e9 / peak}
    pack_bytes = n * (dims[0] * 4.0 + binding.packed_stride_words(dims[0]) * 4.0 + 4.0)
    kernels["pack_features"] = {"ms": pack_ms, "GBps": pack_bytes / (pack_ms * 1e-3) / 1e9,
                                "frac_of_hbm_peak": pack_bytes / (pack_ms * 1e-3) / 1e9 / peak}
    achieved = kernels["spmm_l%d" % dom]["GBps_cached_model"]
    dom_name = kernels["spmm_l%d" % dom]["kernel"]
    dom_key = "%s/%s/%s/l%d" % (dom_name, spec.name, kernels["spmm_l%d" % dom]["zeta_format"], dom)
    roofline = {"kernel": "%s (layer %d: %d -> %d columns)" % (dom_name, dom, dims[dom], dims[dom + 1]),
                "bound": "hbm", "achieved": achieved, "peak": peak, "peak_kind": "%s copy bandwidth" % peak_kind,
                "unit": "GB/s", "frac": achieved / peak, "traffic": traffic_record(dom_key),
                "algorithmic_bytes": kernels["spmm_l%d" % dom]["bytes_cached_model"],
                "note": "byte rows (i8 / i8h) halve the DRAM traffic of the 256-column aggregations and leave them bound by "
                        "the per-chunk chain of hand-offs (tcgen05 products, the default) or by instruction issue (the fp32 "
                        "FMA stream, extras.spmm_fma_stream_ms), not HBM; with fp16 rows (--zeta-format 4) the same layer is "
                        "HBM-bound: see extras.spmm_fp16_rows_ms and kernels.*",
                "model": "per launch: 8 B per stored entry (column, value) + rowptr + node weights + output + every "
                         "operand row once + one operand row per further stored entry whose source is not among the "
                         "highest-degree rows an ideal 126 MB cache would hold"}

    # the same launch against the gather alone (no arithmetic): how close the kernel is to what the memory system can do
    go = extras.get("gather_only_ms")
    if isinstance(go, dict) and str(kernels["spmm_l%d" % dom]["row_bytes"]) in go:
        g_ms = go[str(kernels["spmm_l%d" % dom]["row_bytes"])]
        roofline["gather_only_ms"] = g_ms
        roofline["gather_only_over_kernel"] = g_ms / spmm_ms[dom]

    cpu = None
    if not args.no_cpu_baseline:
        try:
            scale = args.cpu_sample_scale or (default_cpu_scale(synth.WORKLOADS[args.config]) if args.scale is None else args.scale)
            v, threads, sample, ms, _, _ = time_oracle(args.config, scale, 3, 1)
            cpu = {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample, "ms_per_step": ms}
        except Exception as exc:      # the oracle is optional equipment for the bench
            cpu = {"value": None, "unit": UNIT, "cores": 0, "kind": "oracle", "sample": "failed: %r" % (exc,)}

    on_tc_layers = [kernels["bitgemm_l%d" % l]["path"].startswith("tcgen05") for l in range(L)]
    dtype = DTYPE_TC if all(on_tc_layers) else (DTYPE if not any(on_tc_layers) else DTYPE_TC + " / " + DTYPE)
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": dtype, "data": "synthetic",
            "config": {"workload": workload_description(spec, n, nnz), "l2": "inputs_exceed_l2",
                       "parallelism": "replicas" if world > 1 else "single-gpu",
                       "zeta_format": {0: "auto", 1: "f32", 2: "i16", 3: "i8", 4: "f16", 5: "i8h"}[args.zeta_format]},
            "clocks": clocks, "e2e": e2e, "gpu_launches": launches, "roofline": roofline, "cpu_baseline": cpu,
            "step_ms_median": statistics.median(per_kernel["step"]), "step_ms_min": min(per_kernel["step"]),
            "extras": extras, "kernels": kernels}
    print(json.dumps(line), flush=True)
    replicas.finish()


def run_sage(args):
    """Side benchmark of the Bi-GraphSAGE layer stack (mean aggregator) on the same workload shapes:
    L layers called one by one through bigcn_sage_layer_forward, hidden activations passed as packed
    bits.  Single GPU; prints one JSON line."""
    import torch
    from paper_2210_13149_b200 import binding, synth

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    dev = torch.device("cuda", 0)
    wl = synth.make_workload(args.config, scale=args.scale, device=dev)
    spec = wl.spec
    dims = list(spec.dims)
    L = len(dims) - 1
    ctx = binding.BiGCN(0)
    G = ctx.mean_adjacency(wl.rowptr, wl.colidx)
    n, nnz = G.n, G.nnz
    W2 = synth.weights(spec.dims, spec.seed + 7, dev)
    bn = wl.bn_layers()
    pairs = []
    for l in range(L):
        bs, a_s = ctx.pack_weights(wl.W[l])
        bnb, a_n = ctx.pack_weights(W2[l])
        pairs.append([bs, a_s, bnb, a_n])
    # calibrate the batch-norm constants layer after layer with the library's own statistics
    layers = []
    sh, sc = ctx.col_stats(wl.X) if bn[0] else (None, None)
    bits, beta = ctx.pack_features(wl.X, sh, sc)
    x_shift, x_scale = sh, sc
    for l in range(L):
        ls = binding.make_layer(dims[l], dims[l + 1], pairs[l][0], pairs[l][1], sh, sc)
        ln = binding.make_layer(dims[l], dims[l + 1], pairs[l][2], pairs[l][3])
        layers.append((ls, ln))
        if l + 1 < L:
            out = ctx.sage_layer_forward(G, ls, ln, bits, beta, want_h=True)
            sh, sc = ctx.col_stats(out["h"]) if bn[l + 1] else (None, None)
            bits, beta = ctx.pack_features(out["h"], sh, sc)
            del out
    del bits, beta

    def step():
        b, be = ctx.pack_features(wl.X, x_shift, x_scale)
        for l in range(L):
            last = l == L - 1
            o = ctx.sage_layer_forward(G, layers[l][0], layers[l][1], b, be, want_h=last,
                                       next_layer=None if last else layers[l + 1][0])
            b, be = o["next_bits"], o["next_beta"]
        return o["h"]

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    sampler = ClockSampler(0)
    sampler.start()
    time.sleep(0.25)
    launches0 = ctx.launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for _ in range(args.steps):
        step()
    ev1.record()
    torch.cuda.synchronize()
    ms = ev0.elapsed_time(ev1) / args.steps
    line = {"metric": "bisage_forward_nodes_per_s", "value": n / (ms * 1e-3), "unit": UNIT, "n_gpus": 1,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": DTYPE, "data": "synthetic",
            "config": {"workload": "Bi-GraphSAGE (mean aggregator) on " + workload_description(spec, n, nnz),
                       "l2": "inputs_exceed_l2", "note": "layer-by-layer calls: pack + per layer 2 bit-GEMMs + 1 aggregation"},
            "clocks": sampler.stop(), "gpu_launches": ctx.launch_count() - launches0}
    print(json.dumps(line), flush=True)


def run_entropy(args):
    """Side benchmark of the binning entropy estimator (Sec. 6.2) on synthetic activations with the shape
    of the largest row of the paper's entropy table: 2,449,029 samples x 128 neurons, 1000 intervals
    (scaled by --scale).  Single GPU; prints one JSON line; the oracle is timed on a bounded sample."""
    import numpy as np
    import torch
    import oracle
    from paper_2210_13149_b200 import binding

    n, d, M = max(1, int(2449029 * (args.scale or 1.0))), 128, 1000
    dev = torch.device("cuda", 0)
    g = torch.Generator(device=dev).manual_seed(2210)
    H = torch.randn((n, d), device=dev, generator=g) * (torch.rand(d, device=dev, generator=g) * 3.8 + 0.2)
    H[:, ::4].clamp_(min=0)                        # every fourth neuron rectified
    ctx = binding.BiGCN(0)
    for _ in range(max(args.warmup, 3)):
        out = ctx.entropy_bins(H, M)
    torch.cuda.synchronize()
    sampler = ClockSampler(0)
    sampler.start()
    time.sleep(0.25)
    launches0 = ctx.launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for _ in range(args.steps):
        out = ctx.entropy_bins(H, M)
    ev1.record()
    torch.cuda.synchronize()
    ms = ev0.elapsed_time(ev1) / args.steps
    peak, peak_kind = load_peaks()
    algo = 2.0 * n * d * 4                          # the matrix is read twice: range pass, histogram pass
    cpu = None
    if not args.no_cpu_baseline:
        ns = min(n, 200000)
        Hs = H[:ns].cpu().numpy()
        t0 = time.perf_counter()
        ref = oracle.entropy_bins(Hs, M)
        dt = time.perf_counter() - t0
        got = ctx.entropy_bins(H[:ns], M)
        assert np.array_equal(got["counts"].cpu().numpy().astype(np.int64), ref.counts)
        cpu = {"value": ns / dt, "unit": "samples/s", "cores": 1, "kind": "oracle",
               "sample": "the first %d samples of the same matrix (counts checked against the GPU's)" % ns}
    line = {"metric": "entropy_estimate_samples_per_s", "value": n / (ms * 1e-3), "unit": "samples/s", "n_gpus": 1,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32 compare + u32 count + f64 log", "data": "synthetic",
            "config": {"workload": "binning entropy estimate, %d samples x %d neurons, %d intervals" % (n, d, M),
                       "l2": "inputs_exceed_l2"},
            "clocks": sampler.stop(), "gpu_launches": ctx.launch_count() - launches0,
            "roofline": {"bound": "hbm", "achieved": algo / (ms * 1e-3) / 1e9, "peak": peak, "peak_kind": "%s copy bandwidth" % peak_kind,
                         "unit": "GB/s", "frac": algo / (ms * 1e-3) / 1e9 / peak, "traffic": None},
            "cpu_baseline": cpu, "H_ind_bits": out["total"].item()}
    print(json.dumps(line), flush=True)


def run_backward(args):
    """Side benchmark of the back-propagation through one binarized layer (Algorithm 1) on the workload's
    graph: the widest hidden layer (c5: 256 -> 256), input gradient included.  Single GPU; one JSON line;
    the oracle is timed on a draw of the same recipe at a small scale."""
    import numpy as np
    import torch
    import oracle
    from paper_2210_13149_b200 import binding, synth

    dev = torch.device("cuda", 0)
    spec = synth.scaled_spec(args.config, args.scale) if args.scale else synth.WORKLOADS[args.config]
    wl = synth.make_workload(args.config, scale=args.scale, device=dev)
    n = wl.n
    dims = [w.shape[0] for w in wl.W] + [wl.W[-1].shape[1]]
    l = max(range(1, len(wl.W)), key=lambda i: dims[i] * dims[i + 1]) if len(wl.W) > 1 else 0
    d_in, d_out = dims[l], dims[l + 1]
    ctx = binding.BiGCN(0)
    G = ctx.normalize_adjacency(wl.rowptr, wl.colidx)
    nnz = G.nnz
    gen = torch.Generator(device=dev).manual_seed(77)
    W = wl.W[l]
    bitsT, alpha = ctx.pack_weights(W)
    layer = binding.make_layer(d_in, d_out, bitsT, alpha)
    bits, beta = ctx.pack_features(torch.randn((n, d_in), device=dev, generator=gen))
    g_out = torch.randn((n, d_out), device=dev, generator=gen) * 0.02
    for _ in range(max(args.warmup, 3)):
        ctx.layer_backward(G, layer, W, bits, beta, g_out)
    torch.cuda.synchronize()
    sampler = ClockSampler(0)
    sampler.start()
    time.sleep(0.25)
    launches0 = ctx.launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for _ in range(args.steps):
        ctx.layer_backward(G, layer, W, bits, beta, g_out)
    ev1.record()
    torch.cuda.synchronize()
    ms = ev0.elapsed_time(ev1) / args.steps
    cpu = None
    if not args.no_cpu_baseline:
        small = synth.make_workload(args.config, scale=min(1.0, 20000.0 / synth.WORKLOADS[args.config].n))
        src, dst = synth.edge_list(small.rowptr, small.colidx)
        g = oracle.normalize_adjacency(small.n, src, dst)
        rng = np.random.default_rng(3)
        F, be = oracle.binarize_rows(rng.standard_normal((small.n, d_in)).astype(np.float32))
        go = (rng.standard_normal((small.n, d_out)) * 0.02).astype(np.float32)
        t0 = time.perf_counter()
        oracle.layer_backward(g, W.cpu().numpy(), F, be, go)
        dt = time.perf_counter() - t0
        cpu = {"value": small.n / dt, "unit": UNIT, "cores": 1, "kind": "oracle",
               "sample": "the same recipe at %d nodes, same layer widths" % small.n}
    flops = 2.0 * 2.0 * n * d_in * d_out                 # the two dense products
    line = {"metric": "bigcn_layer_backward_nodes_per_s", "value": n / (ms * 1e-3), "unit": UNIT, "n_gpus": 1,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": "Algorithm 1 for layer %d (%d -> %d) on " % (l, d_in, d_out) + workload_description(spec, n, nnz),
                       "l2": "inputs_exceed_l2"},
            "clocks": sampler.stop(), "gpu_launches": ctx.launch_count() - launches0,
            "dense_products_TFLOPs_if_alone": flops / (ms * 1e-3) / 1e12, "cpu_baseline": cpu}
    print(json.dumps(line), flush=True)


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.model == "sage":
        run_sage(args)
    elif args.model == "entropy":
        run_entropy(args)
    elif args.model == "backward":
        run_backward(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

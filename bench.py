#!/usr/bin/env python
"""Benchmark of the three-layer sparse SpMM on B200.

One "step" = one pass of the whole hot path over the OPT-13B-shaped workload (hidden size 5120):
W of 5120x5120, 20480x5120 and 5120x20480 at 50 % per-row magnitude sparsity, each multiplied by X
with N = 8, 16 and 32 -- nine SpMM launches, captured as ONE CUDA graph on ONE stream, in N-major
order.  Every launch reads its own device copy of its weight matrix, so a step streams 918 MB,
seven times the 126 MB L2, and no weight byte is touched twice within a step.

Prints ONE JSON line (rank 0).  `value` is the achieved HBM rate of that single-stream step:
algorithmic bytes of a step (compressed W blob + X + Y of every launch) / device time of a step,
inputs resident in HBM; the median of five timed blocks of `--steps` steps each.  Beside it:
  per_shape      every one of the nine launches timed alone (a graph of that launch over rotating
                 cold copies of its matrix), with the same-shape cuBLAS fp16 GEMM timed the same way;
  three_streams  the same step with its nine independent products forked over three streams;
  extra          the decoder-block stack at hidden 7168, 9216x9216 at N = 64 and the 11008x4096
                 sparsity row (40-70 %), same protocol;
  format_conversion  host encode and device pack+upload seconds per matrix;
  e2e            the same metric through tl3_spmm_host_async (host X and Y, copies in the timed region).

`--impl reference` times the CPU oracle (oracle/, unmodified) on the same metric and workload, on a
bounded sample per step.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2607_08786_b200 import dist, workloads as wl  # noqa: E402

METRIC = "spmm_achieved_hbm_gbs"
UNIT = "GB/s"
WORKLOAD = "config2_opt13b_shapes_50pct_N8_16_32"
# dram__bytes_read.sum + dram__bytes_write.sum of one launch / its algorithmic bytes, from an ncu
# capture of one 8192 x 8192 launch (86 MB blob; the benchmark's 133 MB blobs are too large to
# capture); traffic grows in proportion to the blob, so the ratio is applied to the bytes of a launch
NCU_TRAFFIC_RATIO = 1.03
N_STREAMS = 3            # for the `three_streams` figure
L2_BYTES = 126e6
BLOCKS = 5               # timed blocks of --steps steps; the median is reported


def log(*a):
    print(*a, file=sys.stderr, flush=True)


def measured_peak_gbs():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


def step_cases(seed_offset: int = 0):
    """Config 2 in launch order: N-major, shapes inside."""
    cases = list(wl.config_cases(2))
    out = []
    for N in (8, 16, 32):
        for c in cases:
            if c.N == N:
                out.append(wl.Case(c.config, c.name, c.M, c.K, c.N, c.seed + seed_offset, c.sparsity, c.kind))
    return out


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except Exception:
                continue
            for name, val in zip(names, f[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------------
def run_reference(args, rank):
    """CPU oracle on the host cores: same metric, bounded sample of the same workload per step."""
    if rank != 0:
        return
    import oracle
    oracle.build()
    sample = [c for c in step_cases() if c.N == 16 and c.M == 5120 and c.K == 5120]   # one matrix, N = 16
    prepared = []
    for c in sample:
        W, X = c.make_W(), c.make_X()
        cont = oracle.encode(W)
        prepared.append((cont, X, cont.nbytes() + X.nbytes + c.M * c.N * 2))

    def step():
        for cont, X, _ in prepared:
            oracle.spmm(cont, X)
    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = (time.perf_counter() - t0) / args.steps
    nbytes = sum(b for _, _, b in prepared)
    value = nbytes / dt / 1e9
    desc = {"value": value, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
            "sample": "5120x5120 at N=16 (1 of the 9 launches of a step), canonical container bytes"}
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample": desc["sample"]},
        "cpu_baseline": desc,
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }), flush=True)


# ------------------------------------------------------------------------------------------------
# Timing helpers shared by the headline run and the sweeps
def _capture(fn):
    """fn() once eagerly (lazy set-up), then captured as a CUDA graph."""
    import torch
    fn()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        fn()
    return g


def _time_replays(g, n, blocks=BLOCKS):
    """Device time of one replay in ms: `blocks` blocks of n replays between two events on the
    launching stream; returns (median, all blocks)."""
    import torch
    for _ in range(3):
        g.replay()
    torch.cuda.synchronize()
    out = []
    for _ in range(blocks):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(torch.cuda.current_stream())
        for _ in range(n):
            g.replay()
        b.record(torch.cuda.current_stream())
        torch.cuda.synchronize()
        out.append(a.elapsed_time(b) / n)
    return float(np.median(out)), out


def _copies_for(nbytes, at_least=2):
    """Device copies needed so that a copy has left the L2 before it is read again."""
    if nbytes > 3 * L2_BYTES:
        return max(1, at_least)
    return max(at_least, min(12, int(np.ceil(3 * L2_BYTES / nbytes))))


class Weights:
    """One encoded weight matrix with several device copies of its packed blob (and of the dense
    matrix for the cuBLAS baseline).  A launch reads the copy bound to the handle when it is
    enqueued or captured, so a captured sequence can walk over the copies."""

    def __init__(self, tl3, case, dev, at_least=2, dense=True):
        import torch
        self.case = case
        W = case.make_W()
        t0 = time.perf_counter()
        self.m = tl3.encode(W)
        self.encode_s = time.perf_counter() - t0
        t0 = time.perf_counter()
        first = self.m.upload(device=dev)
        torch.cuda.synchronize()
        self.upload_s = time.perf_counter() - t0            # device pack on the host + H2D copy
        self.bytes = self.m.device_bytes()
        self.blobs = [first] + [first.clone() for _ in range(_copies_for(self.bytes, at_least) - 1)]
        self.dense = []
        if dense:
            d0 = torch.from_numpy(W).to(dev)
            self.dense = [d0] + [d0.clone() for _ in range(min(len(self.blobs), _copies_for(W.nbytes, at_least)) - 1)]
        self.W = W
        self.stats = self.m.stats()
        # the same container built by the CUDA encoder (window classification, scans, pairing, chain
        # emission on the GPU; the copy of the arrays back to the host is inside the time)
        self.device_encode_s, self.device_encode_identical, self.device_pack_s, self.device_pack_identical = None, None, None, None
        self.device_convert_s, self.device_convert_identical = None, None
        if dense:
            enc, pack, conv = [], [], []
            for _ in range(2):                               # best of two: the first call of a kind pays for the module load
                t0 = time.perf_counter()
                md = tl3.Matrix.encode_on_device(self.dense[0])
                enc.append(time.perf_counter() - t0)
                self.device_encode_identical = all(np.array_equal(md.canonical(n), self.m.canonical(n))
                                                   for n in ("pdd_bytes", "tile_dir", "res_rho", "chain_len"))
                # ... and packed for the kernel by the CUDA packer (layout pass, blob pass, the copy of
                # the canonical arrays to the device inside the time)
                t0 = time.perf_counter()
                blob_d = md.upload_packed_on_device(device=dev)
                torch.cuda.synchronize()
                pack.append(time.perf_counter() - t0)
                self.device_pack_identical = bool(torch.equal(blob_d, first))
                del blob_d
                md.close()
                # ... and the whole conversion without a host copy of the container: dense W on the
                # device -> packed blob on the device (encode, layout pass, blob pass)
                t0 = time.perf_counter()
                mo = tl3.Matrix.encode_on_device(self.dense[0], device_only=True)
                blob_o = mo.upload_packed_on_device(device=dev)
                torch.cuda.synchronize()
                conv.append(time.perf_counter() - t0)
                self.device_convert_identical = bool(torch.equal(blob_o, first))
                del blob_o
                mo.close()
            self.device_encode_s, self.device_pack_s, self.device_convert_s = min(enc), min(pack), min(conv)

    def spmm(self, i, X, Y, ws, stream=None):
        self.m.bind(self.blobs[i % len(self.blobs)])
        self.m.spmm(X, Y, workspace=ws, stream=stream)

    def close(self):
        self.m.close()
        self.blobs, self.dense = [], []


def _time_alone(wt, X, Y, ws, reps=20):
    """One launch timed alone: a graph that runs it once on every device copy in turn (each copy is
    cold again when its turn comes), replayed; and the cuBLAS GEMM of the dense matrix the same way.
    Returns (spmm us, dense us or None)."""
    import torch
    n = len(wt.blobs)
    us = _time_replays(_capture(lambda: [wt.spmm(i, X, Y, ws) for i in range(n)]), reps)[0] * 1e3 / n
    dus = None
    if wt.dense:
        out = torch.empty_like(Y)
        nd = len(wt.dense)
        dus = _time_replays(_capture(lambda: [torch.matmul(d, X, out=out) for d in wt.dense]), reps)[0] * 1e3 / nd
    return us, dus


def _row(wt, N, us, dus, peak):
    c = wt.case
    nbytes = wt.bytes + c.K * N * 2 + c.M * N * 2
    st = wt.stats
    r = {"M": c.M, "K": c.K, "N": N, "sparsity": c.sparsity, "us": round(us, 2), "gbs": round(nbytes / us / 1e3, 1),
         "frac_measured": round(nbytes / us / 1e3 / peak, 4), "frac_nominal_8tbs": round(nbytes / us / 1e3 / 8000.0, 4),
         "dense_equiv_tflops": round(2.0 * c.M * c.K * N / us / 1e6, 2),
         "bytes_over_dense": round(st["device_bytes"] / (2 * c.M * c.K), 4)}
    if dus is not None:
        r["dense_gemm_us"] = round(dus, 2)
        r["speedup_vs_dense"] = round(dus / us, 3)
    return r


# ------------------------------------------------------------------------------------------------
def run_ours(args, rank, local_rank, world):
    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    from paper_2607_08786_b200 import build, tl3
    build.build_library()
    tl3.lib()
    dev = torch.device("cuda", local_rank)
    peak, peak_kind = measured_peak_gbs()

    cases = step_cases(dist.rank_seed_offset(rank))
    # One Weights object per shape; launch j of a step (N index j // 3) reads device copy j // 3 of
    # its shape, so no weight byte is touched twice within a step, and the per-shape timing walks
    # over all copies of the shape.
    t_setup = time.time()
    weights, conversion = {}, []
    for c in cases:
        key = (c.M, c.K)
        if key in weights:
            continue
        wt = weights[key] = Weights(tl3, c, dev, at_least=3)
        st = wt.stats
        conversion.append({"M": c.M, "K": c.K, "host_encode_s": round(wt.encode_s, 3), "device_pack_upload_s": round(wt.upload_s, 3),
                           "gpu_encode_s": round(wt.device_encode_s, 3), "gpu_encode_identical": wt.device_encode_identical,
                           "gpu_pack_s": round(wt.device_pack_s, 3), "gpu_pack_identical": wt.device_pack_identical,
                           "gpu_convert_on_device_s": round(wt.device_convert_s, 4), "gpu_convert_identical": wt.device_convert_identical,
                           "canonical_bytes": st["canonical_bytes"], "device_bytes": st["device_bytes"],
                           # shares of the non-zeros by layer: the canonical container, and the device image that
                           # actually streams (its chains are cut after three code words, the tails travel as
                           # Residual entries, and its delta bytes include the zero padding of short chains)
                           "canonical_shares": {"tc": round(st["n_tc"] / st["nnz"], 4), "sf": round(st["n_sf"] / st["nnz"], 4),
                                                "res": round(st["n_res"] / st["nnz"], 4), "dummy": round(st["n_dummy"] / st["nnz"], 4)},
                           "device_shares": {"tc": round(st["n_tc"] / st["nnz"], 4), "sf_coded": round(st["dev_n_sf"] / st["nnz"], 4),
                                             "res_entries": round(st["dev_n_res"] / st["nnz"], 4),
                                             "dummy_and_padding_bytes": round(st["dev_n_dummy"] / st["nnz"], 4)}})
        log(f"[rank {rank}] {c.M}x{c.K}: nnz {st['nnz']} TC {st['n_tc']/st['nnz']:.4f} SF {st['n_sf']/st['nnz']:.4f} "
            f"RES {st['n_res']/st['nnz']:.4f} dummies {st['n_dummy']/st['nnz']:.4f} blob {st['device_bytes']/1e6:.1f} MB "
            f"({st['device_bytes']/(2*c.M*c.K):.4f} x dense, canonical {st['canonical_bytes']/(2*c.M*c.K):.4f}) "
            f"| device image: coded SF {st['dev_n_sf']/st['nnz']:.4f} RES entries {st['dev_n_res']/st['nnz']:.4f} "
            f"dummy+padding bytes {st['dev_n_dummy']/st['nnz']:.4f} | "
            f"encode {wt.encode_s:.2f} s, pack+upload {wt.upload_s:.2f} s, {len(wt.blobs)} device copies")
    launches = []
    for j, c in enumerate(cases):
        wt = weights[(c.M, c.K)]
        X = c.make_X()
        launches.append(dict(case=c, wt=wt, copy=j // 3, X=torch.from_numpy(X).to(dev), Xh=X,
                             Y=torch.empty((c.M, c.N), dtype=torch.float16, device=dev), ws=wt.m.new_workspace(c.N),
                             bytes=wt.bytes + X.nbytes + c.M * c.N * 2, flops=2.0 * c.M * c.K * c.N))
    torch.cuda.synchronize()
    log(f"[rank {rank}] setup {time.time() - t_setup:.1f} s")

    def call(L, stream=None):
        L["wt"].spmm(L["copy"], L["X"], L["Y"], L["ws"], stream=stream)

    def step_serial():
        for L in launches:
            call(L)

    # The nine products of a step do not depend on each other; forked over N_STREAMS streams inside
    # the graph a kernel takes over SMs as the CTAs of a kernel on another stream leave.  Reported
    # as `three_streams`, beside the one-stream headline.
    side_streams = [torch.cuda.Stream(device=dev) for _ in range(N_STREAMS - 1)]

    def forked(calls):
        def run():
            cur = torch.cuda.current_stream()
            ev = torch.cuda.Event()
            ev.record(cur)
            for s in side_streams:
                s.wait_event(ev)
            for i, fn in enumerate(calls):
                st = cur if i % N_STREAMS == 0 else side_streams[i % N_STREAMS - 1]
                with torch.cuda.stream(st):
                    fn(st)
            for s in side_streams:
                done = torch.cuda.Event()
                done.record(s)
                cur.wait_event(done)
        return run

    graph = _capture(step_serial)
    graph3 = _capture(forked([(lambda st, L=L: call(L, st)) for L in launches]))
    stream = torch.cuda.current_stream()
    for _ in range(max(args.warmup, 3)):
        graph.replay()
    torch.cuda.synchronize()
    for L in launches:
        assert L["wt"].m.status(L["ws"]) == tl3.OK

    # ---- timed region: BLOCKS blocks of exactly K steps each, device time, max over ranks
    sampler = ClockSampler(local_rank)
    sampler.start()
    blocks = []
    for _ in range(BLOCKS):
        dist.barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(args.steps):
            graph.replay()
        e1.record(stream)
        torch.cuda.synchronize()
        dist.barrier()
        blocks.append(dist.max_over_ranks(e0.elapsed_time(e1), device=dev) / args.steps)
    clocks = sampler.stop()
    for L in launches:
        word = L["wt"].m.status_word(L["ws"])
        assert word == 0, f"kernel status word {word:#x} for {L['case'].name}"
    ms_step = float(np.median(blocks))
    step_bytes = sum(L["bytes"] for L in launches)
    total_bytes = dist.sum_over_ranks(step_bytes, device=dev)
    value = total_bytes / (ms_step * 1e-3) / 1e9
    ms3 = _time_replays(graph3, max(10, min(args.steps, 100)))[0]

    # ---- same-shape dense fp16 GEMM (cuBLAS through torch.matmul): the same step, same two graphs
    outs = [torch.empty_like(L["Y"]) for L in launches]
    dense_calls = [(lambda st=None, i=i, L=L: torch.matmul(L["wt"].dense[L["copy"] % len(L["wt"].dense)], L["X"], out=outs[i]))
                   for i, L in enumerate(launches)]
    nrep = max(10, min(args.steps, 100))
    dense_ms = _time_replays(_capture(lambda: [fn() for fn in dense_calls]), nrep)[0]
    dense_ms3 = _time_replays(_capture(forked(dense_calls)), nrep)[0]

    # ---- every launch of the step timed alone, and its dense GEMM the same way
    table = []
    for L in launches:
        us, dus = _time_alone(L["wt"], L["X"], L["Y"], L["ws"])
        table.append(_row(L["wt"], L["case"].N, us, dus, peak))
        assert L["wt"].m.status(L["ws"]) == tl3.OK

    # ---- end to end through the C ABI with host buffers (pinned), copies inside the timed region
    e2e_bufs = []
    for L in launches:
        c = L["case"]
        Xp = torch.from_numpy(L["Xh"]).pin_memory()
        Yp = torch.empty((c.M, c.N), dtype=torch.float16).pin_memory()
        dX = torch.empty(c.K * ((c.N + 7) // 8 * 8) * 2, dtype=torch.uint8, device=dev)
        dY = torch.empty(c.M * c.N * 2, dtype=torch.uint8, device=dev)
        e2e_bufs.append((Xp.numpy(), Yp.numpy(), dX, dY))
    # the nine products are independent: each is enqueued (copy in, kernel, copy out) on one of three
    # streams in turn, so the copies of one overlap the kernel of another, and the step ends when all
    # three streams have drained
    e2e_streams = [torch.cuda.Stream(device=dev) for _ in range(3)]

    def step_e2e():
        for i, (L, (Xp, Yp, dX, dY)) in enumerate(zip(launches, e2e_bufs)):
            L["wt"].m.bind(L["wt"].blobs[L["copy"]])
            L["wt"].m.spmm_host_async(Xp, Yp, dX, dY, L["ws"], stream=e2e_streams[i % 3])
        for s in e2e_streams:
            s.synchronize()

    def timed_e2e(step_fn):
        for _ in range(3):
            step_fn()
        out = []
        for _ in range(3):
            dist.barrier()
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            for _ in range(args.steps):
                step_fn()
            torch.cuda.synchronize()
            out.append(dist.max_over_ranks((time.perf_counter() - t0) / args.steps, device=dev))
        return float(np.median(out)), out

    e2e_eager_s, _ = timed_e2e(step_e2e)
    # The same nine calls (copy in, kernel, copy out each, three streams) captured once as a CUDA
    # graph -- tl3_spmm_host_async only enqueues, so a caller can do that -- and replayed per step; the
    # step ends when the host has waited for the stream, i.e. when every Y is in host memory.
    def e2e_call(st, L, bufs):
        Xp, Yp, dX, dY = bufs
        L["wt"].m.bind(L["wt"].blobs[L["copy"]])
        L["wt"].m.spmm_host_async(Xp, Yp, dX, dY, L["ws"], stream=st)

    e2e_graph = _capture(forked([(lambda st, L=L, b=b: e2e_call(st, L, b)) for L, b in zip(launches, e2e_bufs)]))

    def step_e2e_graph():
        e2e_graph.replay()
        torch.cuda.current_stream().synchronize()

    for (Xp, Yp, dX, dY) in e2e_bufs:
        Yp[:] = 0
    e2e_s, e2e_blocks = timed_e2e(step_e2e_graph)
    e2e_value = total_bytes / e2e_s / 1e9
    h2d = sum(L["Xh"].nbytes for L in launches)
    d2h = sum(L["case"].M * L["case"].N * 2 for L in launches)
    # the host-buffer path must give the same numbers as the device path
    for L, (Xp, Yp, dX, dY) in zip(launches[:2], e2e_bufs[:2]):
        assert np.array_equal(Yp.view(np.uint16), L["Y"].cpu().numpy().view(np.uint16))

    if rank != 0:
        return
    ll = launches[0]["wt"].m.last_launch()

    # ---- CPU baseline: the oracle as it stands on a bounded sample (rank 0, N = 1 only), its encode
    #      time beside the library's, and the parity of that launch while the oracle's result is at hand
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        import oracle
        oracle.build()
        L0 = [L for L in launches if L["case"].M == 5120 and L["case"].K == 5120 and L["case"].N == 16][0]
        c, W, X = L0["case"], L0["wt"].W, L0["Xh"]
        t0 = time.perf_counter()
        cont = oracle.encode(W)
        oracle_encode_s = time.perf_counter() - t0
        oracle.spmm(cont, X)
        ts = []
        for _ in range(3):
            t0 = time.perf_counter()
            Yo = oracle.spmm(cont, X)
            ts.append(time.perf_counter() - t0)
        nb = cont.nbytes() + X.nbytes + c.M * c.N * 2
        cpu = {"value": nb / min(ts) / 1e9, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
               "sample": "5120x5120 at N=16 (1 of the 9 launches of a step), best of 3",
               "us": min(ts) * 1e6, "oracle_encode_s": round(oracle_encode_s, 3)}
        call(L0)
        torch.cuda.synchronize()
        Yg = L0["Y"].cpu().numpy().astype(np.float64)
        Yref, bound = oracle.dense_fp64(W, X)
        assert np.all(np.abs(Yg - Yref) <= oracle.tolerance(bound)), "GPU result outside tolerance"
        assert np.all(np.abs(Yo.view(np.float16).astype(np.float64) - Yref) <= oracle.tolerance(bound))

    # ---- further workloads, same protocol (one GPU only: they would stretch a multi-rank run)
    extra = None
    if world == 1 and not args.no_extra:
        for wt in weights.values():
            wt.close()
        launches_info = [(L["case"], L["bytes"]) for L in launches]
        del launches, e2e_bufs, outs, dense_calls, graph, graph3
        torch.cuda.empty_cache()
        extra = run_extra(tl3, dev, peak)
    else:
        launches_info = [(L["case"], L["bytes"]) for L in launches]

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f16xf16->f32", "data": "synthetic",
        "config": {"workload": WORKLOAD, "launches_per_step": len(launches_info), "order": "N-major",
                   "l2": "inputs larger than L2: every launch of a step reads its own copy of W, a step streams 918 MB",
                   "bytes_per_step": step_bytes, "graph": True, "streams": 1, "ctas": ll["ctas"], "smem_bytes": ll["smem_bytes"],
                   "timed": f"median of {BLOCKS} blocks of {args.steps} steps", "blocks_ms_per_step": [round(b, 5) for b in blocks]},
        "clocks": clocks,
        "gpu_launches": len(launches_info) * args.steps * BLOCKS,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": e2e_s * 1e3, "blocks_ms_per_step": [round(b * 1e3, 4) for b in e2e_blocks],
                "how": "tl3_spmm_host_async x 9 on three streams captured as one CUDA graph; per step: replay, then wait for the stream "
                       "(every Y in pinned host memory); host wall clock",
                "eager_ms_per_step": e2e_eager_s * 1e3},
        "roofline": {"bound": "hbm", "achieved": step_bytes / (ms_step * 1e-3) / 1e9, "peak": peak, "unit": "GB/s",
                     "frac": step_bytes / (ms_step * 1e-3) / 1e9 / peak,
                     "peak_kind": f"of {peak_kind}", "frac_nominal_8tbs": step_bytes / (ms_step * 1e-3) / 1e9 / 8000.0,
                     "traffic": NCU_TRAFFIC_RATIO * step_bytes / len(launches_info),
                     "kernel": "tl3_spmm_kernel",
                     "step_us_over_launches": ms_step * 1e3 / len(launches_info),
                     "algorithmic_bytes_per_launch": step_bytes / len(launches_info),
                     "note": "nine back-to-back launches on one stream: bytes of a step / device time of a step, launch "
                             "overlap (programmatic dependent launch) included; per_shape has every launch alone"},
        "cpu_baseline": cpu,
        "dense_fp16_gemm": {"ms_per_step": dense_ms, "speedup_of_spmm": dense_ms / ms_step,
                            "note": "cuBLAS through torch.matmul on the dense masked W, same nine products, same one-stream graph"},
        "three_streams": {"ms_per_step": ms3, "value": step_bytes / (ms3 * 1e-3) / 1e9, "frac": step_bytes / (ms3 * 1e-3) / 1e9 / peak,
                          "dense_ms_per_step": dense_ms3,
                          "note": "the nine independent products forked over three streams inside the graph"},
        "per_shape_note": "each launch alone: a CUDA graph that runs it once on every device copy of its matrix in turn "
                          "(a copy has left the L2 before its next turn), replayed; cuBLAS the same way",
        "per_shape": table,
        "format_conversion": conversion,
        "extra": extra,
    }
    print(json.dumps(out), flush=True)


def _stack(tl3, dev, peak, reps=20):
    """The four linear layers of one decoder block at hidden 7168 / FFN 28672, N = 16, back to back
    on one stream as one CUDA graph (the block's 778 MB of weights evict themselves from the L2)."""
    import torch
    cases = list(wl.config_cases(5))
    wts = [Weights(tl3, c, dev, at_least=1) for c in cases]
    Xs = [torch.from_numpy(c.make_X()).to(dev) for c in cases]
    Ys = [torch.empty((c.M, c.N), dtype=torch.float16, device=dev) for c in cases]
    wss = [wt.m.new_workspace(c.N) for wt, c in zip(wts, cases)]
    us = _time_replays(_capture(lambda: [wt.spmm(0, X, Y, ws) for wt, X, Y, ws in zip(wts, Xs, Ys, wss)]), reps)[0] * 1e3
    dus = _time_replays(_capture(lambda: [torch.matmul(wt.dense[0], X, out=Y) for wt, X, Y in zip(wts, Xs, Ys)]), reps)[0] * 1e3
    for wt, ws in zip(wts, wss):
        assert wt.m.status(ws) == tl3.OK
    flops = sum(2.0 * c.M * c.K * c.N for c in cases)
    nbytes = sum(wt.bytes + c.K * c.N * 2 + c.M * c.N * 2 for wt, c in zip(wts, cases))
    out = {"layers": [f"{c.M}x{c.K}" for c in cases], "N": 16, "us": round(us, 2), "gbs": round(nbytes / us / 1e3, 1),
           "frac_measured": round(nbytes / us / 1e3 / peak, 4), "dense_equiv_tflops": round(flops / us / 1e6, 2),
           "dense_stack_us": round(dus, 2), "speedup_vs_dense": round(dus / us, 3),
           "host_encode_s": [round(wt.encode_s, 2) for wt in wts], "device_pack_upload_s": [round(wt.upload_s, 2) for wt in wts],
           "res_share": [round(wt.stats["n_res"] / wt.stats["nnz"], 4) for wt in wts]}
    for wt in wts:
        wt.close()
    del Xs, Ys, wss
    torch.cuda.empty_cache()
    return out


def _point(tl3, dev, peak, case, verify_rows=0):
    """One (matrix, N) point timed alone, with its dense GEMM; optionally a sample of rows against float64."""
    import torch
    wt = Weights(tl3, case, dev)
    X = case.make_X()
    Xd = torch.from_numpy(X).to(dev)
    Y = torch.empty((case.M, case.N), dtype=torch.float16, device=dev)
    ws = wt.m.new_workspace(case.N)
    us, dus = _time_alone(wt, Xd, Y, ws)
    assert wt.m.status(ws) == tl3.OK
    row = _row(wt, case.N, us, dus, peak)
    st = wt.stats
    row.update({"name": case.name, "sf_share": round(st["n_sf"] / st["nnz"], 4), "res_share": round(st["n_res"] / st["nnz"], 4),
                "host_encode_s": round(wt.encode_s, 2), "device_pack_upload_s": round(wt.upload_s, 2),
                # the container on disk: as the paper stores it, and with the Residual layer and the
                # value array in their compact forms (the kernel streams the device image above)
                "container_over_dense": round(st["canonical_bytes"] / (2 * case.M * case.K), 4),
                "container_compact_over_dense": round(st["canonical_bytes_compact_all"] / (2 * case.M * case.K), 4)})
    if verify_rows:
        rows = np.random.default_rng(case.seed).choice(case.M, size=verify_rows, replace=False)
        Wr = wt.W[rows].astype(np.float64)
        ref, bound = Wr @ X.astype(np.float64), np.abs(Wr) @ np.abs(X.astype(np.float64))
        err = np.abs(Y[torch.from_numpy(rows).to(dev)].cpu().numpy().astype(np.float64) - ref)
        row["verified_rows"] = int(verify_rows)
        row["max_err_over_tol"] = round(float(np.max(err / (2e-3 * bound + 1e-3))), 4)
    wt.close()
    del Xd, Y, ws
    torch.cuda.empty_cache()
    return row


def run_extra(tl3, dev, peak):
    """What the headline line carries beside the OPT-13B step."""
    extra = {"stack_hidden7168_n16": _stack(tl3, dev, peak)}
    extra["c4_9216x9216_n64"] = _point(tl3, dev, peak, [c for c in wl.config_cases(4) if c.M == 9216 and c.K == 9216 and c.N == 64][0], verify_rows=64)
    extra["c3_11008x4096_n16_by_sparsity"] = [_point(tl3, dev, peak, c, verify_rows=64) for c in wl.config_cases(3) if c.M == 11008]
    return extra


def run_single(args):
    """A few launches of one SpMM (for profilers): `--single M K N [--launches L] [--sparsity S]`."""
    import torch
    from paper_2607_08786_b200 import build, tl3
    build.build_library()
    M, K, N = args.single
    case = wl.Case(0, f"single_{M}x{K}_n{N}", M, K, N, 6, args.sparsity, "magnitude")
    m = tl3.encode(case.make_W())
    m.upload()
    Xd = torch.from_numpy(case.make_X()).cuda()
    ws = m.new_workspace(N)
    Y = torch.empty((M, N), dtype=torch.float16, device="cuda")
    for _ in range(args.launches):
        m.spmm(Xd, Y, workspace=ws)
    torch.cuda.synchronize()
    print(json.dumps({"single": case.name, "launches": args.launches, "status": m.status(ws), **m.last_launch(),
                      "device_bytes": m.device_bytes()}), flush=True)


def run_sweep(args):
    """Extra measurements beside the headline: `--sweep n|sparsity|stack|large|small`.  One JSON line per point."""
    import torch
    from paper_2607_08786_b200 import build, tl3
    build.build_library()
    peak, _ = measured_peak_gbs()
    dev = torch.device("cuda", 0)

    def emit(row, label):
        print(json.dumps({"sweep": args.sweep, "point": label, **row}), flush=True)

    if args.sweep == "n":
        for N in (8, 16, 32, 64, 128, 256, 512):
            emit(_point(tl3, dev, peak, wl.Case(4, "n_sweep", 9216, 9216, N, 4000, 0.5, "row_scaled")), f"N={N}")
    elif args.sweep == "large":
        # the shape of the comparison against cuBLAS in the paper's Introduction (M/K/N = 66K/16K/32), and N = 16
        for N in (32, 16):
            emit(_point(tl3, dev, peak, wl.Case(0, f"paper_66k_16k_n{N}", 65536, 16384, N, 6000, 0.5, "magnitude"), verify_rows=64), f"65536x16384_n{N}")
    elif args.sweep == "small":
        for M, K, N in ((1024, 1024, 8), (2048, 2048, 16), (4096, 4096, 16), (4096, 4096, 32), (7168, 7168, 16), (8192, 8192, 16)):
            emit(_point(tl3, dev, peak, wl.Case(0, f"small_{M}x{K}_n{N}", M, K, N, 7000 + M // 128, 0.5, "magnitude")), f"{M}x{K}_n{N}")
    elif args.sweep == "sparsity":
        for case in wl.config_cases(3):
            emit(_point(tl3, dev, peak, case), case.name)
    elif args.sweep == "stack":
        print(json.dumps({"sweep": "stack", **_stack(tl3, dev, peak)}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extra", action="store_true", help="leave out the further workloads (stack, N = 64, sparsity row)")
    ap.add_argument("--single", type=int, nargs=3, metavar=("M", "K", "N"), help="run a few launches of one shape and exit")
    ap.add_argument("--launches", type=int, default=3)
    ap.add_argument("--sweep", choices=["n", "sparsity", "stack", "large", "small"], help="extra measurements; one JSON line per point")
    ap.add_argument("--sparsity", type=float, default=0.5)
    args = ap.parse_args()
    if args.single:
        run_single(args)
        return
    if args.sweep:
        run_sweep(args)
        return
    rank, local_rank, world = dist.env_world()
    if args.impl == "reference":
        run_reference(args, rank)
        return
    if world > 1:
        dist.init_process_group("nccl")
    run_ours(args, rank, local_rank, world)
    if world > 1:
        import torch.distributed as td
        td.destroy_process_group()


if __name__ == "__main__":
    main()

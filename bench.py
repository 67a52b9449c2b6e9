#!/usr/bin/env python
"""Benchmark of the CO3 hot path on B200: batched client encode + parameter-server decode-aggregate.

One step = one training round of the workload: every client's gradient is corrected, converted,
entropy-coded (memory updated) in one batched `co3_encode` call, then all streams are decoded and
averaged by `co3_decode_aggregate`.  Prints one JSON line (the README lists the keys).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config 3] [--no-table]

The headline workload is the largest configuration that fits one GPU (100 clients x 11.2 M elements); the
other configurations are measured in the same run with fewer steps and reported under roofline.per_config.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "co3_encode_decode_aggregate_throughput"
UNIT = "gradient elements/s"
NOMINAL_HBM_GBS = 8000.0     # the peak the metric is defined against; fractions of the measured copy rate beside it
# dram__bytes_read.sum + dram__bytes_write.sum per element of one launch, from the ncu captures summarised under
# profiles/ (taken on a 10-client case; traffic grows in proportion to the elements of a launch).  None: the kernel
# has changed since its counters were taken.
NCU_TRAFFIC_BYTES_PER_ELEMENT = {"pack": 12.511, "decode": 1.050, "convert": 12.579}   # decode: per client and element
# l1tex__data_pipe_lsu_wavefronts_mem_shared.sum per decoded symbol of decode_kernel, from ncu captures on small cases
# (10 clients side by side; 32 clients in batches).  The decoder is bound by this pipe, which takes one wavefront per
# cycle and SM: the table look-ups of a warp collide in the 32 banks.
NCU_DECODE_SMEM_WAVEFRONTS_PER_SYMBOL = {"side_by_side": 0.2534, "batched": 0.2736}
RANK_SEED_STRIDE = 100_000   # ranks draw their synthetic clients from disjoint seed ranges
L2_BYTES = 126e6


def max_over_ranks(ms: float, world: int, device) -> float:
    """Step time of the job: the slowest rank's."""
    if world <= 1:
        return ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def elements_per_step(n_elem: int, clients_per_rank: int, world: int) -> int:
    """Whole-job work of one step: every rank encodes and aggregates its own clients (weak scaling)."""
    return n_elem * clients_per_rank * world


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        return float(p["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return 6650.0, "fallback (6.65 TB/s copy rate, no MEASURED_PEAKS.json)"


def workload(cfg_idx: int, clients_override=None, elements_override=None, cell=None, part_b=False):
    """(cfg, sizes, fmts, clients) of configuration 1..5.  cell: for the sweep (4) one of its cells, default the
    first; part_b: the 8-client half of configuration 5."""
    import co3_inputs as ci
    cfg = ci.config(cfg_idx)
    if part_b:
        cfg = dict(cfg, name=cfg["name"] + "_8clients", sizes=cfg["part_b"]["sizes"], clients=cfg["part_b"]["clients"])
    if elements_override is not None and len(cfg["sizes"]) == 1:
        cfg = dict(cfg, sizes=(int(elements_override),))
    if "cells" in cfg:      # the sweep config: one cell
        cell = cfg["cells"][0] if cell is None else cell
        cfg = dict(cfg, fmt=cell["fmt"], beta=(cell["beta"],), decay=cell["decay"],
                   name="%s_fmt%d%d_beta%g_decay%g" % ((cfg["name"],) + tuple(cell["fmt"]) + (cell["beta"], cell["decay"])))
    sizes = cfg["sizes"]
    E, M = cfg["fmt"]
    fmts = []
    for k in range(len(sizes)):
        s, inv = ci.scale_for(E, M, cfg["beta"][k], cfg["alpha"][k])
        fmts.append((E, M, 0, s, inv))
    clients = cfg["clients"] if clients_override is None else clients_override
    return cfg, sizes, fmts, clients


def make_grads(cfg, sizes, n_clients, stride, rnd, device, rank=0):
    """[n_clients * stride] fp32 on `device`: client u, layer k i.i.d. GenNorm(beta_k, alpha_k)."""
    import torch
    import co3_inputs as ci
    out = torch.zeros(n_clients * stride, dtype=torch.float32, device=device)
    for u in range(n_clients):
        seed = ci.client_round_seed(cfg["seed"] + RANK_SEED_STRIDE * rank, u, rnd)
        off = u * stride
        for k, n in enumerate(sizes):
            out[off:off + n] = ci.gennorm(int(n), float(cfg["beta"][k]), float(cfg["alpha"][k]),
                                          seed * 1_000_003 + k, device,
                                          cfg.get("outlier_frac", 0.0), cfg.get("outlier_mult", 1.0))
            off += n
    return out


class ClockSampler:
    """nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q, "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            f = [x.strip() for x in r.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for name, val in zip(names, f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------------ the oracle on the host
PIECE_ELEMS = 131072     # 64 chunks: pieces of layers are independent work items (chunks are coded independently)


def oracle_pieces(cfg, sizes, fmts, n_workers):
    """The layer layout cut into pieces of at most PIECE_ELEMS elements and dealt to n_workers lists, longest first."""
    pieces = []
    for k, n in enumerate(sizes):
        for lo in range(0, int(n), PIECE_ELEMS):
            pieces.append((k, min(PIECE_ELEMS, int(n) - lo), float(cfg["beta"][k]), float(cfg["alpha"][k]),
                           tuple(fmts[k]), int(cfg["seed"]) * 1_000_003 + 977 * k + lo // PIECE_ELEMS))
    pieces.sort(key=lambda p: -p[1])
    loads = [0] * n_workers
    lists = [[] for _ in range(n_workers)]
    for p in pieces:
        w = loads.index(min(loads))
        lists[w].append(p)
        loads[w] += p[1]
    return lists


def _oracle_worker(wid, pieces, decay, reps, n_iter, start, out_q):
    """One host process: convert + encode of `reps` clients' share of every piece it owns, then the decode-aggregate
    over those clients, n_iter times, through the unchanged oracle.  Inputs and codes are made before the clock starts."""
    import torch
    torch.set_num_threads(1)
    import co3_inputs as ci
    import oracle
    data = []
    for (k, n, beta, alpha, fmt, seed) in pieces:
        E, M, _, s, inv = fmt
        ofmt = oracle.Fmt(E, M, 0, s, inv)
        gs = [ci.gennorm(n, beta, alpha, seed + 7919 * r).numpy() for r in range(reps)]
        r0 = oracle.convert(gs[0], np.zeros(n, dtype=np.float32), decay, ofmt)
        code = oracle.code_build(oracle.histogram(r0["sym"]), ofmt)
        data.append((n, ofmt, code, gs, [np.zeros(n, dtype=np.float32) for _ in range(reps)]))
    out_q.put(("ready", wid, None))
    start.wait()
    per_iter = []
    for _ in range(n_iter):
        t0 = time.perf_counter()
        elems = 0
        for (n, ofmt, code, gs, ms) in data:
            streams = []
            for g, m in zip(gs, ms):
                r = oracle.convert(g, m, decay, ofmt)
                st, s = oracle.encode(r["sym"], [n], [code])
                assert st == oracle.OK
                streams.append(s)
            st, _ = oracle.decode_aggregate(streams, [n], [ofmt], [code])
            assert st == oracle.OK
            elems += n * reps
        per_iter.append((elems, time.perf_counter() - t0))
    out_q.put(("done", wid, per_iter))


def oracle_parallel(cfg, sizes, fmts, n_workers, reps, n_iter):
    """The oracle over independent (layer piece) items on n_workers host processes (started with `spawn`, so that a
    CUDA context in this process is not inherited).  Returns per iteration (elements, seconds), the seconds being the
    slowest worker's busy time."""
    import multiprocessing as mp
    ctx = mp.get_context("spawn")
    lists = [l for l in oracle_pieces(cfg, sizes, fmts, n_workers) if l]
    start, q = ctx.Event(), ctx.Queue()
    procs = [ctx.Process(target=_oracle_worker, args=(w, lists[w], float(cfg["decay"]), reps, n_iter, start, q), daemon=True)
             for w in range(len(lists))]
    for p in procs:
        p.start()
    got = {}
    try:
        for _ in procs:
            tag, wid, _ = q.get(timeout=600)
            assert tag == "ready"
        start.set()
        for _ in procs:
            tag, wid, per_iter = q.get(timeout=1200)
            assert tag == "done"
            got[wid] = per_iter
    finally:
        for p in procs:
            p.join(timeout=30)
            if p.is_alive():
                p.kill()
    out = []
    for i in range(n_iter):
        out.append((sum(got[w][i][0] for w in got), max(got[w][i][1] for w in got)))
    return out, len(procs)


def host_cores() -> int:
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:
        return max(1, os.cpu_count() or 1)


def cpu_baseline(cfg, sizes, fmts, clients, seconds_per_iter=4.0):
    """The oracle, as it stands, on one core and on all host cores, on a bounded sample of the workload."""
    n = int(sum(sizes))
    cores = host_cores()
    one, _ = oracle_parallel(cfg, sizes, fmts, 1, 2, 2)
    one_rate = one[-1][0] / one[-1][1]
    reps = int(min(32, max(2, round(seconds_per_iter * cores * one_rate / n))))
    allc, used = oracle_parallel(cfg, sizes, fmts, cores, reps, 2)
    rate = allc[-1][0] / allc[-1][1]
    what = "full layer layout (%d elements) in pieces of <= %d elements: convert + encode + decode-aggregate" % (n, PIECE_ELEMS)
    return {"value": rate, "unit": UNIT, "cores": used, "kind": "oracle",
            "sample": "%d of %d clients, %s, %.1f s on %d processes (second of two passes)" % (reps, clients, what, allc[-1][1], used),
            "one_core": {"value": one_rate, "unit": UNIT, "cores": 1,
                         "sample": "2 of %d clients, %s, %.1f s" % (clients, what, one[-1][1])}}


def run_reference(args):
    """The CPU oracle as the reference arm, on all host cores: each step pushes a bounded sample of the workload
    (some of its clients, the full layer layout) through convert + encode + decode-aggregate."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg, sizes, fmts, clients = workload(args.config)
    if len(sizes) == 1 and sizes[0] > 20_000_000:      # a long flat vector: its leading 20 M elements
        sizes = (20_000_000,)
    n = int(sum(sizes))
    cores = host_cores()
    # size the sample so that the whole run stays near two minutes: one core does about 6e6 elements/s
    budget_s = 100.0 / max(1, args.steps + args.warmup)
    reps = int(min(32, max(1, budget_s * cores * 6.0e6 / n)))
    per_iter, used = oracle_parallel(cfg, sizes, fmts, cores, reps, args.warmup + args.steps)
    timed = per_iter[args.warmup:]
    elems, secs = sum(e for e, _ in timed), sum(s for _, s in timed)
    value = elems / secs
    sample = "%d of %d clients, layer layout of %d elements in pieces of <= %d, per step, on %d processes" % (
        reps, clients, n, PIECE_ELEMS, used)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * secs / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": cfg["name"], "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": used, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------------ our arm
class Timed:
    """K repetitions of a function on a stream, timed with CUDA events.  Workloads smaller than a few L2 sizes get
    an L2 flush (a 512 MB buffer rewritten) before every repetition and one event pair per repetition."""

    def __init__(self, stream, dev, flush: bool):
        import torch
        self.torch, self.stream, self.flush = torch, stream, flush
        self.buf = torch.empty(512 << 20, dtype=torch.uint8, device=dev) if flush else None

    def run(self, fn, k: int) -> float:
        torch = self.torch
        if not self.flush:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(self.stream)
            for i in range(k):
                fn(i)
            e1.record(self.stream)
            torch.cuda.synchronize()
            return e0.elapsed_time(e1)
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(k)]
        for i in range(k):
            self.buf.fill_(i & 0xff)
            ev[i][0].record(self.stream)
            fn(i)
            ev[i][1].record(self.stream)
        torch.cuda.synchronize()
        return sum(a.elapsed_time(b) for a, b in ev)


def kernel_rows(prof, calls, alg_bytes, peak):
    """Per-kernel averages from a profile read that covered `calls` calls."""
    rows = {}
    for name, (n, tot) in prof.items():
        if n == 0:
            continue
        avg_ms = tot / n
        r = {"launches_per_call": n / calls, "avg_ms": avg_ms, "ms_per_call": tot / calls}
        if name in alg_bytes:
            gbs = alg_bytes[name] / 1e9 / (tot / calls * 1e-3)
            r.update(algorithmic_gb_per_call=alg_bytes[name] / 1e9, achieved_gbs=gbs, frac_of_measured=gbs / peak,
                     frac_of_8tbs=gbs / NOMINAL_HBM_GBS)
        rows[name] = r
    return rows


def measure(cfg, sizes, fmts, clients, dev, rank, world, steps, warmup, peak, headline=False):
    """Times the step (encode call + decode-aggregate call) of one workload, then each call's kernels in a second
    pass with an event pair around every launch."""
    import torch
    import torch.distributed as dist
    import paper_2204_08211_b200 as co3
    from paper_2204_08211_b200.session import Co3Session

    sess = Co3Session(sizes, fmts, clients, cfg["decay"], dev)
    n_rounds = 2
    grads = [make_grads(cfg, sizes, clients, sess.stride, r, dev, rank) for r in range(n_rounds)]
    mems = sess.new_client_buffer()
    # setup (untimed, as the paper reuses the fitted parameters for many rounds): one code per layer from the
    # symbol statistics of the first round, summed over the clients
    hist = sess.histogram(grads[0], sess.new_client_buffer())
    sess.set_codes_from_weights(hist)
    stream = torch.cuda.current_stream()
    fit = bool(cfg.get("fit_per_round"))
    sym_step = sess.new_client_buffer(torch.uint8) if fit else None
    n_local = sess.n_elem * clients
    flush = 8.0 * n_local < 4 * L2_BYTES
    timed = Timed(stream, dev, flush)

    def encode_on(g):
        if fit:     # the code is fitted to this round's symbols: convert + histogram, Huffman tables built on
                    # the device from that histogram, then pack from the symbols; nothing goes through the host
            sess.histogram(g, mems, stream, sym_step, to_host=False)
            sess.set_codes_from_histogram_device(stream)
            sess.encode_symbols(sym_step, stream)
        else:
            sess.encode(g, mems, stream)

    def step_on(g):
        encode_on(g)
        return sess.decode_aggregate(stream)

    def check():
        er = sess.encode_results()
        dr = sess.decode_result()
        if (er["status"] != co3.OK).any() or dr["status"][0] != co3.OK:
            raise RuntimeError("device status: encode %s decode %s" % (er["status"], dr["status"]))
        if fit and sess.fit_result()["status"][0] != co3.OK:
            raise RuntimeError("device status: code build %s" % sess.fit_result()["status"])
        return er, dr

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    for i in range(warmup):
        step_on(grads[i % n_rounds])
    barrier()
    check()

    sampler = ClockSampler(dev.index or 0) if (headline and rank == 0) else None
    if sampler:
        sampler.start()
    barrier()
    ms = timed.run(lambda i: step_on(grads[(warmup + i) % n_rounds]), steps)
    barrier()
    clocks = sampler.stop() if sampler else None
    er, dr = check()
    ms = max_over_ranks(ms, world, dev)

    # ---- small workloads are launch-bound: the same step once more as a CUDA-graph replay
    graph_ms = None
    if flush and world == 1:
        try:
            side = torch.cuda.Stream(device=dev)
            graph = torch.cuda.CUDAGraph()

            def captured():     # the calls take the capturing stream (the current one)
                if fit:
                    sess.histogram(grads[0], mems, None, sym_step, to_host=False)
                    sess.set_codes_from_histogram_device(None)
                    sess.encode_symbols(sym_step, None)
                else:
                    sess.encode(grads[0], mems, None)
                sess.decode_aggregate(None)

            with torch.cuda.graph(graph, stream=side):
                captured()
            torch.cuda.synchronize()
            for _ in range(3):
                graph.replay()
            graph_ms = timed.run(lambda i: graph.replay(), steps) / steps
            check()
        except Exception as exc:     # a capture that fails must not take the benchmark down
            graph_ms = "capture failed: %s" % str(exc)[:120]
            torch.cuda.synchronize()

    # ---- each call on its own: the encode calls, then the decode calls, timed as wholes
    enc_call_ms = timed.run(lambda i: encode_on(grads[(warmup + i) % n_rounds]), steps) / steps
    dec_call_ms = timed.run(lambda i: sess.decode_aggregate(stream), steps) / steps
    check()

    # ---- per-kernel times: the same calls again, an event pair around every launch
    co3.co3_profile_enable(True)
    timed.run(lambda i: encode_on(grads[(warmup + i) % n_rounds]), steps)
    prof_enc = co3.co3_profile_read()
    timed.run(lambda i: sess.decode_aggregate(stream), steps)
    prof_dec = co3.co3_profile_read()
    co3.co3_profile_enable(False)
    check()

    container = float(er["container_bytes"].astype(np.float64).sum())
    bits = float(er["payload_bits"].astype(np.float64).sum())
    # algorithmic bytes: what the method must move.  Encode: g and m in, m and the container out (fitted every
    # round: g, m in, m and symbols out; then symbols in, container out).  Decode: containers in, average out.
    alg_enc = (12.0 if not fit else 14.0) * n_local + container
    alg_dec = 4.0 * sess.n_elem + container
    enc_rows = kernel_rows(prof_enc, steps, {"pack": (1.0 if fit else 12.0) * n_local + container, "convert": 13.0 * n_local}, peak)
    dec_rows = kernel_rows(prof_dec, steps, {"decode": alg_dec}, peak)
    enc_ms, dec_ms = enc_call_ms, dec_call_ms
    enc_sum = sum(r["ms_per_call"] for r in enc_rows.values())
    dec_sum = sum(r["ms_per_call"] for r in dec_rows.values())
    launches = sum(r["launches_per_call"] for r in enc_rows.values()) + sum(r["launches_per_call"] for r in dec_rows.values())

    def call_row(ms_call, alg):
        gbs = alg / 1e9 / (ms_call * 1e-3)
        return {"ms": ms_call, "algorithmic_gb": alg / 1e9, "achieved_gbs": gbs, "frac_of_measured": gbs / peak,
                "frac_of_8tbs": gbs / NOMINAL_HBM_GBS, "elements_per_s": n_local / (ms_call * 1e-3)}

    row = {
        "workload": cfg["name"], "clients": clients, "elements_per_client": sess.n_elem, "layers": sess.n_seg,
        "format": "[1,%d,%d]" % tuple(cfg["fmt"]), "decay": cfg["decay"], "steps": steps,
        "ms_per_step": ms / steps, "elements_per_s": n_local * world * steps / (ms * 1e-3),
        "effective_gbs": (alg_enc + alg_dec) * world / 1e9 / (ms / steps * 1e-3),
        "mean_code_bits": bits / n_local, "container_bits_per_element": 8.0 * container / n_local,
        "index_and_padding_bits_per_element": (8.0 * container - bits) / n_local,
        "l2": "L2 flushed before every step (512 MB rewritten)" if flush else
              "inputs larger than L2 (%.0f MB of gradients and memory per step)" % (8.0 * n_local / 1e6),
        "encode_call": dict(call_row(enc_ms, alg_enc), kernels=enc_rows, kernels_sum_ms=enc_sum,
                            note="the call that leaves the containers in place, timed as a whole; `kernels` come from a "
                                 "further pass with an event pair around every launch (their sum carries the events' cost "
                                 "and loses the overlap of dependent launches)"),
        "decode_call": dict(call_row(dec_ms, alg_dec), kernels=dec_rows, kernels_sum_ms=dec_sum),
        "launches_per_step": launches,
    }
    if graph_ms is not None:
        row["cuda_graph_replay_ms_per_step"] = graph_ms
    if "compact" in enc_rows:   # the slots pack leaves behind are read and written once more: not algorithmic
        row["encode_call"]["non_algorithmic_gb"] = 2.0 * container / 1e9
    state = dict(sess=sess, grads=grads, mems=mems, stream=stream, step_on=step_on, check=check, barrier=barrier,
                 clocks=clocks, er=er, timed=timed, n_local=n_local, container=container, fit=fit)
    return row, state


def standalone_kernels(state, cfg, clients, steps, warmup, peak):
    """Calls outside the step, over the same data, each kernel timed by its own event pair."""
    import torch
    import co3_inputs as ci
    import paper_2204_08211_b200 as co3
    sess, grads, stream, timed, n_local = state["sess"], state["grads"], state["stream"], state["timed"], state["n_local"]
    dev = sess.device
    out = {}

    def row(gb, n, tot, calls):
        gbs = gb / (tot / calls * 1e-3)
        return {"ms_per_call": tot / calls, "launches_per_call": n / calls, "algorithmic_gb_per_call": gb,
                "achieved_gbs": gbs, "frac_of_measured": gbs / peak, "frac_of_8tbs": gbs / NOMINAL_HBM_GBS,
                "note": "stand-alone call over the same data, outside the timed step"}

    def timed_calls(fn, kind):
        for i in range(warmup):
            fn(i)
        torch.cuda.synchronize()
        co3.co3_profile_enable(True)
        timed.run(fn, steps)
        p = co3.co3_profile_read()
        co3.co3_profile_enable(False)
        return p[kind]

    sym_buf = sess.new_client_buffer(torch.uint8)
    mems_k1 = sess.new_client_buffer()

    def conv(hist_buf, sym):
        def f(i):
            st = co3.co3_convert(grads[i % 2], mems_k1, sess.decay, sess.fmts, sess.segs, sess.n_seg, sess.n_elem,
                                 clients, sess.stride, sym, hist_buf, sess.res_enc, sess.workspace, stream)
            if st != co3.OK:
                raise RuntimeError("co3_convert: " + co3.co3_status_string(st))
        return f

    n, tot = timed_calls(conv(None, sym_buf), "convert")
    out["convert_standalone"] = row(13.0 * n_local / 1e9, n, tot, steps)
    n, tot = timed_calls(conv(sess.hist, sym_buf), "convert")
    out["convert_hist_standalone"] = row(13.0 * n_local / 1e9, n, tot, steps)

    def dry(i):     # the symbol statistics alone: gradient and memory in, nothing but 256 counters per layer out
        st = co3.co3_histogram(grads[i % 2], mems_k1, sess.decay, sess.fmts, sess.segs, sess.n_seg, sess.n_elem,
                               clients, sess.stride, sess.hist, sess.res_enc, sess.workspace, stream)
        if st != co3.OK:
            raise RuntimeError("co3_histogram: " + co3.co3_status_string(st))

    n, tot = timed_calls(dry, "convert")
    out["histogram_standalone"] = row(8.0 * n_local / 1e9, n, tot, steps)
    if (sess.encode_results()["status"] != co3.OK).any():
        raise RuntimeError("device status after co3_convert / co3_histogram")
    del sym_buf

    # the data-driven refit of every layer's multiplier (moments of v = g + decay * m, then the per-layer fit), on
    # a copy of the formats so that the timed configuration is not disturbed
    tab, beta0, dbeta = ci.scale_log_table([tuple(cfg["fmt"])])
    d_tab = torch.from_numpy(tab).to(dev)
    fmts_fit = sess.fmts.clone()

    def fit(i):
        st = co3.co3_fit_scale(grads[i % 2], mems_k1, sess.decay, fmts_fit, sess.segs, sess.n_seg, sess.n_elem,
                               clients, sess.stride, d_tab, None, 1, tab.shape[1], beta0, dbeta, None, sess.res_fit,
                               sess.workspace, stream)
        if st != co3.OK:
            raise RuntimeError("co3_fit_scale: " + co3.co3_status_string(st))

    n, tot = timed_calls(fit, "fit")
    out["fit_scale_standalone"] = row(8.0 * n_local / 1e9, n, tot, steps)
    if sess.fit_result()["status"][0] != co3.OK:
        raise RuntimeError("device status after co3_fit_scale")
    del mems_k1

    # one client's stream alone (the parameter server of a single user, U = 1)
    ghat_buf = torch.empty(sess.n_elem, dtype=torch.float32, device=dev)

    def dec1(i):
        st = co3.co3_decode(sess.streams[:sess.capacity], sess.capacity, sess.fmts, sess.codes, sess.segs, sess.n_seg,
                            sess.n_elem, ghat_buf, None, sess.workspace, sess.res_dec, stream=stream)
        if st != co3.OK:
            raise RuntimeError("co3_decode: " + co3.co3_status_string(st))

    n, tot = timed_calls(dec1, "decode")
    one_client_bytes = 4.0 * sess.n_elem + float(state["er"]["container_bytes"][0])
    out["decode_one_client"] = row(one_client_bytes / 1e9, n, tot, steps)
    if sess.decode_result()["status"][0] != co3.OK:
        raise RuntimeError("device status after co3_decode")
    return out


def uniform_symbol_decode(dev, steps, warmup, peak):
    """Decoding when the chunks' payloads do not fit the decoder's shared-memory staging pool: symbols uniform over
    the 239 symbols of [1,4,3] (7.9 bit each), 11.2 M per client, one and ten clients."""
    import torch
    import paper_2204_08211_b200 as co3
    from paper_2204_08211_b200.session import Co3Session
    n = 11_181_642
    out = {}
    for clients in (1, 10):
        sess = Co3Session([n], [(4, 3, 0, 1.0, 1.0)], clients, 0.9, dev)
        valid = np.array([c | (sg << 7) for sg in (0, 1) for c in range(120) if not (sg and c == 0)], dtype=np.uint8)
        rng = np.random.default_rng(0)
        sym = torch.from_numpy(valid[rng.integers(0, valid.size, size=clients * sess.stride)]).to(dev)
        hist = np.zeros((1, 256), dtype=np.uint64)
        hist[0, valid] = 1000
        sess.set_codes_from_weights(hist)
        sess.encode_symbols(sym)
        for _ in range(warmup):
            sess.decode_aggregate()
        torch.cuda.synchronize()
        er = sess.encode_results()
        if (er["status"] != co3.OK).any():
            raise RuntimeError("device status (uniform symbols): %s" % er["status"])
        co3.co3_profile_enable(True)
        for _ in range(steps):
            sess.decode_aggregate()
        n_l, tot = co3.co3_profile_read()["decode"]
        co3.co3_profile_enable(False)
        if sess.decode_result()["status"][0] != co3.OK:
            raise RuntimeError("device status after decode (uniform symbols)")
        gb = (4.0 * n + float(er["container_bytes"].astype(np.float64).sum())) / 1e9
        gbs = gb / (tot / n_l * 1e-3)
        out["decode_uniform_symbols_%dclient%s" % (clients, "s" if clients > 1 else "")] = {
            "ms_per_call": tot / n_l, "launches_per_call": 1.0, "algorithmic_gb_per_call": gb, "achieved_gbs": gbs,
            "frac_of_measured": gbs / peak, "frac_of_8tbs": gbs / NOMINAL_HBM_GBS,
            "mean_code_bits": float(er["payload_bits"].astype(np.float64).sum()) / (clients * n),
            "note": "payloads read in place from global memory (they exceed the staging pool); 11.2 M symbols per client"}
        del sess, sym
    return out


def end_to_end(state, clients, steps, world, dev):
    """Pinned host gradients in, averaged gradient out, every step, through the same calls."""
    import torch
    sess, grads, stream, step_on, barrier = state["sess"], state["grads"], state["stream"], state["step_on"], state["barrier"]
    host_g = torch.empty(clients * sess.stride, dtype=torch.float32, pin_memory=True)
    host_g.copy_(grads[0])
    host_avg = torch.empty(sess.n_elem, dtype=torch.float32, pin_memory=True)
    # two device buffers and a copy stream: the upload of step i + 1 runs while step i computes and downloads
    dev_g = grads       # the two rounds' device buffers are overwritten by the uploads
    copy_stream = torch.cuda.Stream(device=dev)
    ready = [torch.cuda.Event() for _ in range(2)]
    free = [torch.cuda.Event() for _ in range(2)]
    e2e_steps = max(2, min(steps, 10))

    def upload(i):
        b = i & 1
        with torch.cuda.stream(copy_stream):
            copy_stream.wait_event(free[b])
            dev_g[b].copy_(host_g, non_blocking=True)
            ready[b].record(copy_stream)

    def e2e_step(i, last):
        b = i & 1
        if not last:
            upload(i + 1)
        stream.wait_event(ready[b])
        host_avg.copy_(step_on(dev_g[b]), non_blocking=True)
        free[b].record(stream)

    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for b in range(2):
        free[b].record(stream)
    upload(0)
    e2e_step(0, True)           # warm-up step, nothing left in flight
    barrier()
    copy_stream.synchronize()
    e0.record(stream)           # every timed step's upload, compute and download lie between e0 and e1
    upload(1)
    for i in range(1, e2e_steps + 1):
        e2e_step(i, i == e2e_steps)
    e1.record(stream)
    barrier()
    e2e_ms = max_over_ranks(e0.elapsed_time(e1), world, dev)
    state["check"]()
    return {"value": sess.n_elem * clients * world * e2e_steps / (e2e_ms * 1e-3), "unit": UNIT, "steps": e2e_steps,
            "ms_per_step": e2e_ms / e2e_steps, "h2d_bytes_per_step": int(4 * clients * sess.stride),
            "d2h_bytes_per_step": int(4 * sess.n_elem)}


def table_workloads():
    """The other configurations, each at full size (the sweep: one cell per format)."""
    import co3_inputs as ci
    out = [workload(1), workload(2)]
    seen = set()
    for cell in ci.config(4)["cells"]:
        if cell["fmt"] not in seen and cell["beta"] == 1.0 and cell["decay"] == 0.9:
            seen.add(cell["fmt"])
            out.append(workload(4, cell=cell))
    out += [workload(5), workload(5, part_b=True)]
    return out


def run_ours(args):
    import gc
    import torch
    import torch.distributed as dist

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    peak, peak_src = load_peaks()

    cfg, sizes, fmts, clients = workload(args.config, args.clients, args.elements)
    row, state = measure(cfg, sizes, fmts, clients, dev, rank, world, args.steps, args.warmup, peak, headline=True)
    alone = standalone_kernels(state, cfg, clients, args.steps, args.warmup, peak)
    e2e = end_to_end(state, clients, args.steps, world, dev)
    n_elem, clocks = state["sess"].n_elem, state["clocks"]
    del state
    gc.collect()
    torch.cuda.empty_cache()
    if world == 1 and not args.no_table:
        alone.update(uniform_symbol_decode(dev, args.steps, args.warmup, peak))
    gc.collect()
    torch.cuda.empty_cache()

    table = []
    if not args.no_table and world == 1:
        for (c2, s2, f2, u2) in table_workloads():
            if c2["name"] == cfg["name"]:
                continue
            r2, st2 = measure(c2, s2, f2, u2, dev, rank, world, args.table_steps, 3, peak)
            table.append(r2)
            del st2
            gc.collect()
            torch.cuda.empty_cache()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel (algorithmic bytes / measured duration)
    kern = dict(row["encode_call"]["kernels"], **row["decode_call"]["kernels"])
    dom = max((k for k in ("pack", "decode", "convert") if k in kern), key=lambda k: kern[k]["ms_per_call"])
    per_elem = NCU_TRAFFIC_BYTES_PER_ELEMENT.get(dom)
    traffic_units = n_elem * clients
    roofline = {"kernel": dom + "_kernel", "bound": "hbm", "achieved": kern[dom]["achieved_gbs"], "peak": peak,
                "unit": "GB/s", "frac": kern[dom]["frac_of_measured"], "frac_of_8tbs": kern[dom]["frac_of_8tbs"],
                "traffic": per_elem * traffic_units if per_elem is not None else None,
                "traffic_unit": "bytes per launch (ncu dram__bytes_read.sum + dram__bytes_write.sum of a smaller launch, scaled by elements)",
                "algorithmic_bytes_per_launch": kern[dom]["algorithmic_gb_per_call"] * 1e9, "peak_source": peak_src,
                "nominal_peak_gbs": NOMINAL_HBM_GBS,
                "timed": "second pass of the same calls with CUDA events around every launch",
                "encode_call": {k: v for k, v in row["encode_call"].items() if k != "kernels"},
                "decode_call": {k: v for k, v in row["decode_call"].items() if k != "kernels"},
                "kernels": dict(kern, **alone),
                "per_config": [row] + table}

    if "decode" in kern and clocks.get("sm_mhz"):
        wf = NCU_DECODE_SMEM_WAVEFRONTS_PER_SYMBOL["batched" if clients > 16 else "side_by_side"]
        sms = torch.cuda.get_device_properties(dev).multi_processor_count
        peak_sym = sms * clocks["sm_mhz"] * 1e6 / wf
        got_sym = n_elem * clients / (kern["decode"]["ms_per_call"] * 1e-3)
        roofline["decode_kernel_shared_memory_pipe"] = {
            "bound": "shared-memory data pipe", "achieved": got_sym, "peak": peak_sym, "unit": "symbols/s",
            "frac": got_sym / peak_sym, "wavefronts_per_symbol": wf,
            "peak_source": "SMs x median SM clock of this run / ncu wavefronts per symbol (one wavefront per cycle and SM)"}

    cpu = None
    if not args.no_cpu_baseline and world == 1:
        cpu = cpu_baseline(cfg, sizes, fmts, clients)

    line = {
        "metric": METRIC, "value": row["elements_per_s"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": row["ms_per_step"], "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": cfg["name"], "clients_per_gpu": clients, "elements_per_client": n_elem,
                   "layers": row["layers"], "format": row["format"], "decay": cfg["decay"],
                   "mean_code_bits": row["mean_code_bits"], "container_bits_per_element": row["container_bits_per_element"],
                   "l2": row["l2"],
                   "code": "fitted every step (convert + histogram, Huffman tables built on the device, pack from symbols)"
                           if cfg.get("fit_per_round") else "fitted once before the timed steps, then reused",
                   "parallelism": "replicas" if world > 1 else "single"},
        "gpu_launches": int(round(row["launches_per_step"] * args.steps)),
        "effective_gbs": row["effective_gbs"],
        "roofline": roofline, "clocks": clocks,
        "e2e": e2e, "cpu_baseline": cpu,
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=3, help="headline workload (1..5); default the largest, 100 clients")
    ap.add_argument("--clients", type=int, default=None, help="override the clients per GPU (profiling small cases)")
    ap.add_argument("--elements", type=int, default=None, help="override the length of a single-layer config (profiling)")
    ap.add_argument("--no-table", action="store_true", help="skip the other configurations")
    ap.add_argument("--table-steps", type=int, default=10)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

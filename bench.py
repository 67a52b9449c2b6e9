#!/usr/bin/env python
"""Benchmark of the CO3 hot path on B200: batched client encode + parameter-server decode-aggregate.

One step = one training round of the workload: every client's gradient is corrected, converted,
entropy-coded (memory updated) in one batched `co3_encode` call, then all streams are decoded and
averaged by `co3_decode_aggregate`.  Prints one JSON line (the README lists the keys).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config 2]
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
# dram__bytes_read.sum + dram__bytes_write.sum of one launch, from the ncu captures summarised under profiles/
# (config 2, 10 clients).  Only meaningful for that workload and for the kernels as they were captured.
NCU_TRAFFIC_BYTES = {"pack": 1397.6e6, "decode": 116.4e6, "convert": 1405.6e6}
RANK_SEED_STRIDE = 100_000   # ranks draw their synthetic clients from disjoint seed ranges


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
    return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


def workload(cfg_idx: int, clients_override=None, elements_override=None):
    import co3_inputs as ci
    cfg = ci.config(cfg_idx)
    if elements_override is not None and len(cfg["sizes"]) == 1:
        cfg = dict(cfg, sizes=(int(elements_override),))
    if "cells" in cfg:      # the sweep config: one representative cell
        cell = cfg["cells"][0]
        cfg = dict(cfg, fmt=cell["fmt"], beta=(cell["beta"],), decay=cell["decay"])
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


# ------------------------------------------------------------------------------------------------ reference arm
def oracle_step(cfg, sizes, fmts, n_clients, codes=None):
    """One bounded sample of the workload through the CPU oracle.  Returns (elements, seconds, codes)."""
    import co3_inputs as ci
    import oracle
    ofmts = [oracle.Fmt(E, M, 0, s, inv) for (E, M, _, s, inv) in fmts]
    offs = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)
    n = int(offs[-1])
    grads = []
    for u in range(n_clients):
        seed = ci.client_round_seed(cfg["seed"], u, 0)
        grads.append(np.concatenate([ci.gennorm(int(sz), float(cfg["beta"][k]), float(cfg["alpha"][k]),
                                                seed * 1_000_003 + k).numpy() for k, sz in enumerate(sizes)]))
    mems = [np.zeros(n, dtype=np.float32) for _ in range(n_clients)]
    if codes is None:        # setup, untimed: fit the per-layer codes on these gradients
        hist = np.zeros((len(sizes), 256), dtype=np.uint64)
        for u in range(n_clients):
            for k in range(len(sizes)):
                r = oracle.convert(grads[u][offs[k]:offs[k + 1]], np.zeros(int(sizes[k]), dtype=np.float32),
                                   cfg["decay"], ofmts[k])
                hist[k] += oracle.histogram(r["sym"])
        codes = [oracle.code_build(hist[k], ofmts[k]) for k in range(len(sizes))]
    t0 = time.perf_counter()
    streams = []
    for u in range(n_clients):
        sym = np.empty(n, dtype=np.uint8)
        for k in range(len(sizes)):
            m = mems[u][offs[k]:offs[k + 1]]
            r = oracle.convert(grads[u][offs[k]:offs[k + 1]], m, cfg["decay"], ofmts[k])
            sym[offs[k]:offs[k + 1]] = r["sym"]
        st, s = oracle.encode(sym, sizes, codes)
        assert st == oracle.OK
        streams.append(s)
    st, avg = oracle.decode_aggregate(streams, sizes, ofmts, codes)
    assert st == oracle.OK
    dt = time.perf_counter() - t0
    return n * n_clients, dt, codes


def run_reference(args):
    """The CPU oracle as the reference arm: each step pushes a bounded sample of the workload (one client, the
    leading layers) through convert + encode + decode-aggregate on one host core."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg, sizes, fmts, clients = workload(args.config)
    # size the sample so that the whole run stays near two minutes: the oracle does about 6e6 elements/s
    budget_s = 100.0 / max(1, args.steps + args.warmup)
    target = max(200_000, int(6.0e6 * budget_s))
    n_layers, acc = 0, 0
    while n_layers < len(sizes) and (n_layers == 0 or acc + sizes[n_layers] <= target):
        acc += sizes[n_layers]
        n_layers += 1
    sub_sizes, sub_fmts = list(sizes[:n_layers]), fmts[:n_layers]
    sub_cfg = dict(cfg, beta=cfg["beta"][:n_layers], alpha=cfg["alpha"][:n_layers])
    _, _, codes = oracle_step(sub_cfg, sub_sizes, sub_fmts, 1, None)
    for _ in range(max(0, args.warmup - 1)):
        oracle_step(sub_cfg, sub_sizes, sub_fmts, 1, codes)
    elems, secs = 0, 0.0
    for _ in range(args.steps):
        e, dt, _ = oracle_step(sub_cfg, sub_sizes, sub_fmts, 1, codes)
        elems += e
        secs += dt
    value = elems / secs
    sample = "1 of %d clients, first %d of %d layers (%d of %d elements) per step" % (
        clients, n_layers, len(sizes), sum(sub_sizes), sum(sizes))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * secs / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": cfg["name"], "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------------ our arm
def run_ours(args):
    import torch
    import torch.distributed as dist
    import paper_2204_08211_b200 as co3
    from paper_2204_08211_b200.session import Co3Session

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    cfg, sizes, fmts, clients = workload(args.config, args.clients, args.elements)
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

    def step_on(g):
        if fit:     # the code is fitted to this round's symbols: convert + histogram, Huffman tables built on
                    # the device from that histogram, then pack from the symbols; nothing goes through the host
            sess.histogram(g, mems, stream, sym_step, to_host=False)
            sess.set_codes_from_histogram_device(stream)
            sess.encode_symbols(sym_step, stream)
        else:
            sess.encode(g, mems, stream)
        return sess.decode_aggregate(stream)

    def step(i):
        step_on(grads[i % n_rounds])

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

    for i in range(args.warmup):
        step(i)
    barrier()
    check()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record(stream)
    for i in range(args.steps):
        step(args.warmup + i)
    e1.record(stream)
    barrier()
    ms = e0.elapsed_time(e1)
    clocks = sampler.stop() if rank == 0 else None
    er, dr = check()
    ms = max_over_ranks(ms, world, dev)
    elems_per_step = elements_per_step(sess.n_elem, clients, world)
    value = elems_per_step * args.steps / (ms * 1e-3)

    # ---- per-kernel times: a second pass of the same steps with an event pair around every launch
    co3.co3_profile_enable(True)
    for i in range(args.steps):
        step(args.warmup + i)
    torch.cuda.synchronize()
    prof = co3.co3_profile_read()
    co3.co3_profile_enable(False)
    launches_per_step = sum(n for n, _ in prof.values()) // args.steps

    # ---- the stand-alone correct + convert + memory kernel (the flow that fits the code between conversion and
    # coding), timed the same way outside the step: with symbols out, and with symbols and histogram out
    sym_buf = sess.new_client_buffer(torch.uint8)
    mems_k1 = sess.new_client_buffer()
    k1 = {}
    for name, hist_buf in (("convert_standalone", None), ("convert_hist_standalone", sess.hist)):
        for i in range(args.warmup + args.steps):
            if i == args.warmup:
                torch.cuda.synchronize()
                co3.co3_profile_enable(True)
            st = co3.co3_convert(grads[i % n_rounds], mems_k1, sess.decay, sess.fmts, sess.segs, sess.n_seg, sess.n_elem,
                                 clients, sess.stride, sym_buf, hist_buf, sess.res_enc, sess.workspace, stream)
            if st != co3.OK:
                raise RuntimeError("co3_convert: " + co3.co3_status_string(st))
        torch.cuda.synchronize()
        k1[name] = co3.co3_profile_read()["convert"]
        co3.co3_profile_enable(False)
    check_enc = sess.encode_results()
    if (check_enc["status"] != co3.OK).any():
        raise RuntimeError("device status after co3_convert: %s" % check_enc["status"])

    # ---- the data-driven refit of every layer's multiplier (moments of v = g + decay * m, then the per-layer fit),
    # on a copy of the formats so that the timed configuration is not disturbed
    import co3_inputs as ci
    tab, beta0, dbeta = ci.scale_log_table([tuple(cfg["fmt"])])
    d_tab = torch.from_numpy(tab).to(dev)
    fmts_fit = sess.fmts.clone()
    for i in range(args.warmup + args.steps):
        if i == args.warmup:
            torch.cuda.synchronize()
            co3.co3_profile_enable(True)
        st = co3.co3_fit_scale(grads[i % n_rounds], mems_k1, sess.decay, fmts_fit, sess.segs, sess.n_seg, sess.n_elem,
                               clients, sess.stride, d_tab, None, 1, tab.shape[1], beta0, dbeta, None, sess.res_fit,
                               sess.workspace, stream)
        if st != co3.OK:
            raise RuntimeError("co3_fit_scale: " + co3.co3_status_string(st))
    torch.cuda.synchronize()
    n_fit, ms_fit = co3.co3_profile_read()["fit"]
    k1["fit_scale_standalone"] = (n_fit // 2, ms_fit)      # two launches (moments, fit) per call
    co3.co3_profile_enable(False)
    if sess.fit_result()["status"][0] != co3.OK:
        raise RuntimeError("device status after co3_fit_scale: %s" % sess.fit_result()["status"])

    # ---- one client's stream alone (the parameter server of a single user, U = 1), same timing method
    sess.encode(grads[0], mems, stream)
    torch.cuda.synchronize()
    ghat_buf = torch.empty(sess.n_elem, dtype=torch.float32, device=dev)
    for i in range(args.warmup + args.steps):
        if i == args.warmup:
            torch.cuda.synchronize()
            co3.co3_profile_enable(True)
        st = co3.co3_decode(sess.streams[:sess.capacity], sess.capacity, sess.fmts, sess.codes, sess.segs, sess.n_seg,
                            sess.n_elem, ghat_buf, None, sess.workspace, sess.res_dec, stream=stream)
        if st != co3.OK:
            raise RuntimeError("co3_decode: " + co3.co3_status_string(st))
    torch.cuda.synchronize()
    k1["decode_one_client"] = co3.co3_profile_read()["decode"]
    co3.co3_profile_enable(False)
    if sess.decode_result()["status"][0] != co3.OK:
        raise RuntimeError("device status after co3_decode")
    one_client_bytes = 4.0 * sess.n_elem + float(sess.encode_results()["container_bytes"][0])

    # ---- end to end: pinned host gradients in, averaged gradient out, every step
    host_g = [torch.empty(clients * sess.stride, dtype=torch.float32).pin_memory() for _ in range(n_rounds)]
    for r in range(n_rounds):
        host_g[r].copy_(grads[r])
    host_avg = torch.empty(sess.n_elem, dtype=torch.float32).pin_memory()
    # two device buffers and a copy stream: the upload of step i + 1 runs while step i computes and downloads
    dev_g = [torch.empty_like(grads[0]) for _ in range(2)]
    copy_stream = torch.cuda.Stream(device=dev)
    ready = [torch.cuda.Event() for _ in range(2)]
    free = [torch.cuda.Event() for _ in range(2)]
    e2e_steps = max(2, min(args.steps, 10))

    def e2e_upload(i):
        b = i & 1
        with torch.cuda.stream(copy_stream):
            copy_stream.wait_event(free[b])
            dev_g[b].copy_(host_g[i % n_rounds], non_blocking=True)
            ready[b].record(copy_stream)

    def e2e_step(i, last):
        b = i & 1
        if not last:
            e2e_upload(i + 1)
        stream.wait_event(ready[b])
        host_avg.copy_(step_on(dev_g[b]), non_blocking=True)
        free[b].record(stream)

    for b in range(2):
        free[b].record(stream)
    e2e_upload(0)
    e2e_step(0, True)           # warm-up step, nothing left in flight
    barrier()
    copy_stream.synchronize()
    e0.record(stream)           # every timed step's upload, compute and download lie between e0 and e1
    e2e_upload(1)
    for i in range(1, e2e_steps + 1):
        e2e_step(i, i == e2e_steps)
    e1.record(stream)
    barrier()
    e2e_ms = e0.elapsed_time(e1)
    e2e_ms = max_over_ranks(e2e_ms, world, dev)
    check()
    e2e_value = elems_per_step * e2e_steps / (e2e_ms * 1e-3)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel (algorithmic bytes / measured duration)
    peak, peak_src = load_peaks()
    n_local = sess.n_elem * clients
    container = float(er["container_bytes"].astype(np.float64).sum())
    alg_bytes = {
        "pack": (1.0 if fit else 12.0) * n_local + container,   # g, m in (or symbols in); m and the container out
        "decode": 4.0 * sess.n_elem + container,     # all containers in; the average out
        "convert": 13.0 * n_local,
    }
    kernels = {}
    for name, (n, tot) in prof.items():
        if n == 0:
            continue
        avg_ms = tot / n
        k = {"launches_per_step": n // args.steps, "avg_ms": avg_ms}
        if name in alg_bytes:
            k["algorithmic_gb_per_launch"] = alg_bytes[name] / 1e9
            k["achieved_gbs"] = alg_bytes[name] / 1e9 / (avg_ms * 1e-3)
            k["frac_of_peak"] = k["achieved_gbs"] / peak
        kernels[name] = k
    for name, (n, tot) in k1.items():
        avg_ms = tot / n
        gb = {"decode_one_client": one_client_bytes, "fit_scale_standalone": 8.0 * n_local}.get(name, alg_bytes["convert"]) / 1e9
        kernels[name] = {"launches_per_step": 0, "avg_ms": avg_ms, "algorithmic_gb_per_launch": gb,
                         "achieved_gbs": gb / (avg_ms * 1e-3), "frac_of_peak": gb / (avg_ms * 1e-3) / peak,
                         "note": "stand-alone call over the same data, outside the timed step"}
    dom = max((k for k in ("pack", "decode") + (("convert",) if fit else ())), key=lambda k: kernels[k]["avg_ms"] * kernels[k]["launches_per_step"])
    roofline = {"kernel": dom + "_kernel", "bound": "hbm", "achieved": kernels[dom]["achieved_gbs"], "peak": peak,
                "unit": "GB/s", "frac": kernels[dom]["frac_of_peak"],
                "traffic": NCU_TRAFFIC_BYTES.get(dom) if (args.config == 2 and clients == 10) else None,
                "traffic_unit": "bytes per launch (ncu dram__bytes_read.sum + dram__bytes_write.sum)",
                "algorithmic_bytes_per_launch": alg_bytes[dom], "peak_source": peak_src,
                "timed": "second pass of the same steps with CUDA events around every launch"}
    bits = float(er["payload_bits"].astype(np.float64).sum())

    # ---- CPU baseline: the oracle on a bounded sample (one client, full layer layout)
    cpu = None
    if not args.no_cpu_baseline:
        n_cpu = min(2, clients)
        elems, secs, _ = oracle_step(cfg, sizes, fmts, n_cpu, None)
        cpu = {"value": elems / secs, "unit": UNIT, "cores": 1, "kind": "oracle",
               "sample": "%d of %d clients, full layer layout (%d elements each): convert + encode + decode-aggregate, "
                         "%.1f s" % (n_cpu, clients, sess.n_elem, secs)}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": cfg["name"], "clients_per_gpu": clients, "elements_per_client": sess.n_elem,
                   "layers": sess.n_seg, "format": "[1,%d,%d]" % tuple(cfg["fmt"]), "decay": cfg["decay"],
                   "mean_code_bits": bits / n_local, "container_bits_per_element": 8.0 * container / n_local,
                   "l2": "inputs larger than L2 (%.0f MB of gradients and memory per step)" % (8.0 * n_local / 1e6),
                   "code": "fitted every step (convert + histogram, Huffman tables built on the device, pack from symbols)" if fit
                           else "fitted once before the timed steps, then reused",
                   "parallelism": "replicas" if world > 1 else "single"},
        "gpu_launches": launches_per_step * args.steps,
        "effective_gbs": (alg_bytes["pack"] + alg_bytes["decode"]) * world / 1e9 / (ms / args.steps * 1e-3),
        "roofline": roofline, "kernels": kernels, "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "steps": e2e_steps, "ms_per_step": e2e_ms / e2e_steps,
                "h2d_bytes_per_step": int(4 * clients * sess.stride), "d2h_bytes_per_step": int(4 * sess.n_elem)},
        "cpu_baseline": cpu,
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=2)
    ap.add_argument("--clients", type=int, default=None, help="override the clients per GPU (profiling small cases)")
    ap.add_argument("--elements", type=int, default=None, help="override the length of a single-layer config (profiling)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

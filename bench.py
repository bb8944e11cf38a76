#!/usr/bin/env python
"""Benchmark of the Deep Gradient Compression hot path on B200.

One *step* is one pass of the whole hot path over one batch of synthetic
gradients: for each of the N_w simulated workers one dgc_compress (clip,
momentum correction, exact top-k selection, emission, masking), then the
decode of the N_w sparse lists into the dense gradient and the SGD step
(dgc_decode_accumulate_sgd: both in one pass; --separate-receive runs
dgc_decode_accumulate and dgc_apply_sgd as two calls).

Headline metric: compressed gradient elements per second (all workers),
inputs resident in HBM.  Beside it: the roofline of the dominant kernel
(algorithmic bytes / its CUDA-event duration / measured copy bandwidth), the
end-to-end number with host buffers, and the CPU oracle timed on this host.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload resnet50|lstm|...]
    python bench.py --impl reference ...     # times the CPU oracle instead

With --gpus N > 1 (under torchrun) every rank runs an independent replica of
the same job on its own GPU (the path has no exchange step on one node: the
N_w workers are simulated in one GPU's memory); time is the max over ranks and
value the sum of all ranks' elements over that time.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_1712_01887_b200 import inputs as I  # noqa: E402

METRIC = "compressed gradient elements/s"
UNIT = "elements/s"
E2E_POOL = 2        # pinned host gradients per worker for the end-to-end leg
LR = 0.01
TRAFFIC_JSON = os.path.join(ROOT, "profiles", "ncu_dram_traffic.json")


def _pool_size(wl, override=None) -> int:
    """Distinct pre-generated gradients per worker: the workload's stated iteration count (10
    for the ResNet-50- and LSTM-shaped sets), so that consecutive steps see fresh gradients;
    --pool overrides it (small profiler captures)."""
    if override:
        return max(1, int(override))
    return max(2, min(int(wl.iterations), 10))


def _ncu_traffic(workload: str, kernel: str):
    """dram__bytes_read.sum + dram__bytes_write.sum of one launch of `kernel` on `workload`,
    from the committed ncu summaries (profiles/ncu_dram_traffic.json); None if not captured."""
    try:
        with open(TRAFFIC_JSON) as f:
            return float(json.load(f)[workload][kernel]["dram_bytes_per_launch"])
    except (OSError, KeyError, ValueError, TypeError):
        return None


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


class ClockSampler:
    """nvidia-smi clocks and throttle reasons, sampled while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "50", "-i", str(self.index)],
                stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        rows = []
        try:
            with open(self.path) as f:
                for line in f:
                    parts = [x.strip() for x in line.split(",")]
                    if len(parts) >= 7 and parts[0].replace(".", "").isdigit():
                        rows.append(parts)
            os.unlink(self.path)
        except Exception:
            pass
        if rows:
            sm = sorted(float(r[0]) for r in rows)
            out["sm_mhz"] = sm[len(sm) // 2]
            out["sm_max_mhz"] = float(rows[0][1])
            out["power_w_max"] = max(float(r[2]) for r in rows if r[2].replace(".", "").isdigit())
            names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
            out["reasons"] = [n for i, n in enumerate(names)
                              if any(r[3 + i].lower().startswith("active") for r in rows)]
            out["samples"] = len(rows)
        return out


def max_over_ranks(value: float, device: str = "cuda") -> float:
    """Replicas only: every rank times its own copy of the job; the job's time is the slowest
    rank's.  No-op without an initialised process group."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(elements_per_rank_step: int, steps: int, world: int, ms_max: float) -> float:
    """Weak scaling: all ranks' elements over the slowest rank's time."""
    return world * elements_per_rank_step * steps / (ms_max * 1e-3)


def _layout(wl):
    return I.packed_layout(wl.numel, align=512)


def _host_gradients(wl, n_workers, rank, pool):
    """pool x n_workers host gradients (numpy), generated once, seeded; a few host threads
    fill them side by side (numpy's generators release the interpreter lock)."""
    from concurrent.futures import ThreadPoolExecutor
    off, L = _layout(wl)

    def one(wi):
        w, i = wi
        a = np.zeros(L, np.float32)
        I.fill(wl, a, off, worker=rank * 1000 + w, iteration=i)
        return a

    jobs = [(w, i) for w in range(n_workers) for i in range(pool)]
    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as ex:
        flat = list(ex.map(one, jobs))
    return off, L, [flat[w * pool:(w + 1) * pool] for w in range(n_workers)]


def _make_pool(wl, n_workers, rank, pool=E2E_POOL):
    """pool x n_workers pinned host gradients (for the modes that copy from the host)."""
    import torch
    off, L, rows = _host_gradients(wl, n_workers, rank, pool)
    hosts = []
    for row in rows:
        out = []
        for a in row:
            t = torch.empty(L, dtype=torch.float32).pin_memory()
            t.numpy()[:] = a
            out.append(t)
        hosts.append(out)
    return off, L, hosts


def measure(args, wl, rank, world, dev, headline):
    """All timings of one workload.  `headline`: also the end-to-end leg, the wire format, the
    timeline and the CPU baseline (the second target workload reports the device timings only)."""
    import torch
    import torch.distributed as dist
    from paper_1712_01887_b200 import binding as B

    NW = args.workers or wl.num_workers
    POOL = _pool_size(wl, args.pool)
    off, L, grads = _host_gradients(wl, NW, rank, POOL)
    total = wl.total
    states = [B.State(wl.numel, wl.num_workers, wl.momentum, wl.clip_threshold, wl.sparsity,
                      sample_ratio=wl.sample_ratio, seed=I.BASE_SEED + w, device=dev)
              for w in range(NW)]
    assert states[0].arena_len == L and np.array_equal(states[0].arena_offset, off)
    nnz = states[0].max_nnz
    pool = [[torch.from_numpy(a).cuda() for a in row] for row in grads]
    hosts = None
    if headline and not args.no_e2e:
        hosts = []
        for row in grads:
            pinned = []
            for a in row[:E2E_POOL]:
                t = torch.empty(L, dtype=torch.float32).pin_memory()
                t.numpy()[:] = a
                pinned.append(t)
            hosts.append(pinned)
    del grads
    out_i = [torch.empty(nnz, dtype=torch.int32, device="cuda") for _ in range(NW)]
    out_v = [torch.empty(nnz, dtype=torch.float32, device="cuda") for _ in range(NW)]
    dense = torch.empty(L, dtype=torch.float32, device="cuda")
    weights = torch.randn(L, dtype=torch.float32, device="cuda")
    ws = torch.empty(max(B.decode_workspace_bytes(NW, L), 4), dtype=torch.uint8, device="cuda")

    # the simulated workers are independent until the decode: their compress calls go round
    # robin over a few streams so that one worker's short selection kernels overlap another
    # worker's streaming pass; the decode waits for all of them
    main_stream = torch.cuda.current_stream()
    NS = max(1, min(args.streams, NW))
    side = [torch.cuda.Stream() for _ in range(NS)] if NS > 1 else [main_stream]
    ev_fork = torch.cuda.Event()
    ev_join = [torch.cuda.Event() for _ in range(NS)]

    def step(t):
        if not args.no_batch:
            # one call for all workers: the library overlaps their kernels itself
            B.compress_batch(states, [pool[w][t % POOL] for w in range(NW)], out_i, out_v)
            receive_side()
            return
        if NS > 1:
            ev_fork.record(main_stream)
            for s_ in side:
                s_.wait_event(ev_fork)
        for w in range(NW):
            states[w].compress(pool[w][t % POOL], out_i[w], out_v[w], stream=side[w % NS])
        if NS > 1:
            for i, s_ in enumerate(side):
                ev_join[i].record(s_)
                main_stream.wait_event(ev_join[i])
        receive_side()

    def receive_side():
        # Alg. 4 aggregation + update lines: the dense gradient is written and the weights are
        # updated; one pass by default, the two separate calls with --separate-receive
        if args.separate_receive:
            B.decode_accumulate(out_i, out_v, dense, ws)
            B.apply_sgd(weights, dense, LR)
        else:
            B.decode_accumulate_sgd(out_i, out_v, dense, weights, LR, ws)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    K, W, R = args.steps, args.warmup, max(1, args.repeats)
    for t in range(W):
        step(t)
    barrier()
    graphs, graph_launches = None, 0
    graphs_used = bool(args.graph)
    eager_step = step
    if args.graph:
        # the whole step captured once per pooled gradient and replayed: every replay is one
        # more iteration on the same buffers (the library keeps its per-call state on the device)
        graphs = []
        for i in range(POOL):
            gr = torch.cuda.CUDAGraph()
            n0 = B.launch_count()
            with torch.cuda.graph(gr):
                step(i)
            graph_launches = B.launch_count() - n0
            graphs.append(gr)

        def step(t):                               # noqa: F811
            graphs[t % POOL].replay()
        for t in range(W):
            step(t)
        barrier()
    sampler = ClockSampler(dev)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    flush = None
    if args.flush_l2:
        # cold-cache variant for working sets that fit the 126 MB L2: a 256 MB buffer is
        # rewritten before every step, outside the per-step event pairs that are summed
        flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    # the timed region, R times: exactly K steps each, bracketed by barrier + synchronize
    rep_ms, launches = [], 0
    t_next = W
    for _ in range(R):
        launches0 = B.launch_count()
        barrier()
        if flush is not None:
            pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
                     for _ in range(K)]
            for q in range(K):
                flush.zero_()
                pairs[q][0].record()
                step(t_next + q)
                pairs[q][1].record()
            barrier()
            ms = sum(a.elapsed_time(b) for a, b in pairs)
        else:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for q in range(K):
                step(t_next + q)
            e1.record()
            barrier()
            ms = e0.elapsed_time(e1)
        t_next += K
        launches = B.launch_count() - launches0
        rep_ms.append(max_over_ranks(ms))
    del flush
    if graphs is not None:
        launches = graph_launches * K              # kernels inside the replayed graphs
        del graphs
    clocks = sampler.stop() if rank == 0 else None
    ms = float(np.median(rep_ms))

    # the same K steps once more with stage events recorded inside every dgc_compress: the
    # dominant kernel's duration for the roofline (the events themselves cost about 3 us per
    # stage, which is why the headline region above runs without them)
    for s in states:
        s.profile_enable(K)
    for t in range(t_next, t_next + K):        # one stream: overlapped kernels cannot be timed
        for w in range(NW):
            states[w].compress(pool[w][t % POOL], out_i[w], out_v[w])
        receive_side()
    torch.cuda.synchronize()
    stage_ms = np.concatenate([s.profile_read(K) for s in states], axis=0)
    kern_ms = stage_ms[:, 2]
    for s in states:
        s.profile_enable(0)

    # compress-only timing, one stream (same states keep evolving): one worker's calls back to
    # back, the deployment the paper describes (one worker per GPU)
    c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    c0.record()
    for t in range(K):
        for w in range(NW):
            states[w].compress(pool[w][t % POOL], out_i[w], out_v[w])
    c1.record()
    torch.cuda.synchronize()
    compress_ms = c0.elapsed_time(c1) / (K * NW)
    # what the last of those calls did, per worker: fallbacks would show here
    last_status = []
    for s_ in states:
        q = s_.status()
        last_status.append({"flags": int(q.flags), "full_select": int(q.full_select_last),
                            "candidates": int(q.candidates_last)})

    # receive side alone: dense decode + SGD (what the step runs) and the fused sparse form
    def _time(fn, reps=20):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        fn()
        torch.cuda.synchronize()
        a.record()
        for _ in range(reps):
            fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / reps

    def _dense_receive():
        B.decode_accumulate(out_i, out_v, dense, ws)
        B.apply_sgd(weights, dense, LR)

    receive = {"decode_plus_sgd_ms": _time(_dense_receive),
               "one_pass_decode_sgd_ms": _time(
                   lambda: B.decode_accumulate_sgd(out_i, out_v, dense, weights, LR, ws)),
               "fused_sparse_decode_sgd_ms": _time(
                   lambda: B.decode_apply_sgd(out_i, out_v, weights, LR, ws))}

    wire = None
    if headline:
        # the paper's wire format (values + 16-bit zero run lengths) of one worker's list
        runs, _vals = B.encode_runlength(out_i[0], out_v[0], L)
        enc_ms = _time(lambda: B.encode_runlength(out_i[0], out_v[0], L), reps=5)
        wire = {"entries": int(runs.numel()), "bytes": int(runs.numel()) * 6,
                "compression_ratio": total * 4 / max(int(runs.numel()) * 6, 1),
                "encode_ms_with_count_readback": enc_ms}

    # end to end through the host-buffer entry point: H2D of every gradient and D2H of the
    # sparse lists inside the timed region
    e2e = None
    if hosts is not None:
        hi = [torch.empty(nnz, dtype=torch.int32).pin_memory() for _ in range(NW)]
        hv = [torch.empty(nnz, dtype=torch.float32).pin_memory() for _ in range(NW)]
        KE = max(1, min(K, args.e2e_steps))

        def e2e_step(t):
            if args.no_batch:
                for w in range(NW):
                    states[w].compress_host(hosts[w][t % E2E_POOL], hi[w], hv[w])
            else:
                B.compress_host_batch(states, [hosts[w][t % E2E_POOL] for w in range(NW)], hi, hv)
            # the lists a receiver would get are on the host now; the receive side runs on the
            # device copies the call also left in the state's output staging
            for w in range(NW):
                out_i[w].copy_(hi[w], non_blocking=True)
                out_v[w].copy_(hv[w], non_blocking=True)
            receive_side()

        e2e_step(0)
        barrier()
        t0 = time.perf_counter()
        for t in range(KE):
            e2e_step(t + 1)
        torch.cuda.synchronize()
        dt = time.perf_counter() - t0
        dt = max_over_ranks(dt)
        e2e = {"value": whole_job_value(NW * total, KE, world, dt * 1e3), "unit": UNIT,
               "h2d_bytes_per_step": NW * (L * 4 + nnz * 8), "d2h_bytes_per_step": NW * nnz * 8,
               "ms_per_step": dt / KE * 1e3, "steps": KE}

    peak, peak_src = _peaks()
    k_ms = float(np.mean(kern_ms))
    alg_bytes = 20.0 * total                       # read g,u,v + write u,v per real element
    achieved = alg_bytes / (k_ms * 1e-3) / 1e9
    compress_bytes = (24.0 if wl.clip_threshold > 0 else 20.0) * total + 16.0 * nnz
    # optional: where on the GPU's clock each worker's kernels ran in one step (the library's
    # timeline aid: first and last block start of every kernel), with the GPU kept busy while
    # the host enqueues the step so that the step runs as it does in the timed loop
    timeline = None
    if args.timeline and headline and rank == 0:
        for s_ in states:
            s_.timeline_enable(True)
        for t in range(3):
            eager_step(t) if graphs_used else step(t)
        torch.cuda.synchronize()
        for s_ in states:
            s_.timeline_read()
        busy = torch.empty(1 << 28, dtype=torch.float32, device="cuda")
        for _ in range(3):
            busy.zero_()
        (eager_step if graphs_used else step)(3)
        torch.cuda.synchronize()
        tl = np.stack([s_.timeline_read().astype(np.int64) for s_ in states])      # [NW, 4, 2]
        t0 = tl[:, :, 0][tl[:, :, 1] > 0].min()
        timeline = {"unit": "us after the step's first block",
                    "kernels": ["sample", "stream", "select", "emit"],
                    "first_last_block_start": [[[round(float(x - t0) / 1e3, 1) for x in k]
                                                for k in w] for w in tl]}
        for s_ in states:
            s_.timeline_enable(False)
        del busy
    # the whole step against the same peak: every worker's compress bytes plus the receive side
    # (lists read, dense gradient written, weights read and written; the two-call form also
    # re-reads the dense gradient)
    recv_bytes = 8.0 * NW * nnz + 4.0 * L + (12.0 if args.separate_receive else 8.0) * L
    step_bytes = NW * compress_bytes + recv_bytes
    step_gbs = step_bytes / (ms / K * 1e-3) / 1e9
    for s_ in states:
        s_.close()
    res = {
        "value": whole_job_value(NW * total, K, world, ms), "ms_per_step": ms / K,
        "repeats": {"n": R, "ms_per_step": [x / K for x in rep_ms],
                    "min": min(rep_ms) / K, "max": max(rep_ms) / K,
                    "reported": "median of the repeats, each exactly `steps` steps"},
        "config": {"workload": wl.name, "tensors": len(wl.shapes), "elements": total,
                   "simulated_workers": NW, "sparsity": wl.sparsity, "momentum": wl.momentum,
                   "clip_threshold": wl.clip_threshold, "sample_ratio": wl.sample_ratio,
                   "nnz_per_worker": nnz,
                   "gradients": f"{POOL} distinct pre-generated gradients per worker, cycled",
                   "compress_call": "dgc_compress per worker on %d streams" % NS if args.no_batch
                   else "dgc_compress_batch (all workers in one call)",
                   "streams": NS,
                   "launch": "cuda graph replay" if args.graph else "stream launches",
                   "receive": "dgc_decode_accumulate + dgc_apply_sgd" if args.separate_receive
                   else "dgc_decode_accumulate_sgd (dense gradient and SGD step in one pass)",
                   "l2": ("flushed: 256 MB rewritten before every step" if args.flush_l2 else
                          "inputs larger than L2 (each worker streams "
                          f"{3 * L * 4 / 1e6:.0f} MB of g,u,v; {NW} workers cycle)"
                          if 3 * L * 4 * NW > 2 * (126 << 20) else
                          f"NOT flushed and L2-resident ({3 * L * 4 * NW / 1e6:.0f} MB of g,u,v "
                          "over all workers): a warm-cache figure, see --flush-l2"),
                   "parallelism": "replicas only" if world > 1 else "1 GPU"},
        "roofline": {"bound": "hbm", "kernel": "k_update_emit", "achieved": achieved,
                     "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "peak_source": peak_src, "frac_of_nominal_8000": achieved / 8000.0,
                     "kernel_ms": k_ms, "kernel_launches": int(kern_ms.size),
                     "kernel_timing": "CUDA events around the kernel inside dgc_compress, on its "
                                      "stream, in an instrumented single-stream repeat of the "
                                      "same K steps",
                     "algorithmic_bytes_per_launch": alg_bytes,
                     "traffic": args.traffic if args.traffic is not None
                     else _ncu_traffic(wl.name, "k_update_emit")},
        "stages_ms": dict(zip(["norm", "sample", "stream", "select", "emit"],
                              [float(x) for x in stage_ms.mean(axis=0)])),
        "compress": {"ms_per_worker": compress_ms, "elements_per_s": total / (compress_ms * 1e-3),
                     "algorithmic_gbs": compress_bytes / (compress_ms * 1e-3) / 1e9,
                     "frac_of_peak": compress_bytes / (compress_ms * 1e-3) / 1e9 / peak,
                     "what": "one dgc_compress alone on one stream (one worker per GPU)",
                     "last_call_status_per_worker": last_status},
        "step": {"algorithmic_bytes": step_bytes, "algorithmic_gbs": step_gbs,
                 "frac_of_peak": step_gbs / peak},
        "timeline": timeline, "receive": receive, "wire_format": wire, "e2e": e2e,
        "gpu_launches": int(launches), "clocks": clocks,
    }
    del pool, out_i, out_v, dense, weights, ws, states
    torch.cuda.empty_cache()
    return res


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_1712_01887_b200 import build
    build.build()

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.cuda.current_device()
    wl = I.workload(args.workload) if args.workload != "sweep" else I.workload("sweep", n=args.n)
    if args.clip is not None:
        wl.clip_threshold = args.clip
    if args.sparsity is not None:
        wl.sparsity = args.sparsity
    head = measure(args, wl, rank, world, dev, headline=True)
    # the second target workload: the LSTM-shaped set (4 workers, clipping on), same step,
    # same clocks sampler, device timings only; part of the default run
    second = None
    plain = (args.workload == "resnet50" and args.clip is None and args.sparsity is None
             and args.workers is None)
    if plain and not args.no_second:
        w2 = I.workload("lstm")
        r2 = measure(args, w2, rank, world, dev, headline=False)
        second = {k: r2[k] for k in ("value", "ms_per_step", "repeats", "config", "roofline",
                                     "stages_ms", "compress", "step", "receive", "gpu_launches",
                                     "clocks")}
        second["unit"] = UNIT
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    cpu = None if args.no_cpu_baseline else cpu_baseline(wl, budget_s=args.cpu_seconds)
    line = {
        "metric": METRIC, "value": head["value"], "unit": UNIT,
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": head["ms_per_step"],
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
    }
    for k in ("config", "repeats", "roofline", "stages_ms", "compress", "step", "timeline",
              "receive", "wire_format", "e2e", "gpu_launches", "clocks"):
        line[k] = head[k]
    line["cpu_baseline"] = cpu
    if second is not None:
        line["lstm"] = second
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


# ----------------------------------------------------------------------------- CPU oracle legs

def _oracle_step_factory(wl, n_workers, pool=E2E_POOL):
    """The same step on the CPU oracle, for `n_workers` simulated workers."""
    from oracle import dgc_oracle as O
    off, L = _layout(wl)
    grads = []
    for w in range(n_workers):
        row = []
        for i in range(pool):
            a = np.zeros(L, np.float32)
            I.fill(wl, a, off, worker=w, iteration=i)
            row.append(a)
        grads.append(row)
    workers = [O.Worker(off, wl.numel, L, wl.num_workers, wl.momentum, wl.clip_threshold,
                        wl.sparsity) for _ in range(n_workers)]
    weights = np.random.default_rng(0).standard_normal(L).astype(np.float32)

    def step(t):
        res = [workers[w].compress(grads[w][t % pool]) for w in range(n_workers)]
        dense = O.decode_accumulate([r.idx for r in res], [r.val for r in res], L)
        O.apply_sgd(weights, dense, LR)

    return step


def cpu_baseline(wl, budget_s=20.0):
    """The oracle as it stands, single thread, on a bounded sample of the workload."""
    nw = min(2, wl.num_workers)
    step = _oracle_step_factory(wl, nw)
    step(0)                                   # first touch / page-in, not timed
    t0 = time.perf_counter()
    n = 0
    while True:
        step(n + 1)
        n += 1
        dt = time.perf_counter() - t0
        if dt >= budget_s or n >= 64:
            break
    return {"value": nw * wl.total * n / dt, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"{n} step(s) of {nw} simulated worker(s) on the full {wl.name} shapes "
                      f"(compress x{nw} + decode + SGD), single thread, {dt:.1f} s",
            "host_cpus": os.cpu_count()}


def run_schedule(args):
    """The warm-up schedule of Sec. 4.1 on one workload (meant for the DeepSpeech-shaped set: 5
    stages of `--stage-iters` iterations at 75 %, 93.75 %, 98.4375 %, 99.6 %, 99.9 % sparsity):
    the same step as the headline benchmark, timed per stage, dgc_set_sparsity between stages."""
    POOL = E2E_POOL
    import torch
    from paper_1712_01887_b200 import build
    build.build()
    from paper_1712_01887_b200 import binding as B
    wl = I.workload(args.workload)
    if args.clip is not None:
        wl.clip_threshold = args.clip
    NW = args.workers or wl.num_workers
    off, L, hosts = _make_pool(wl, NW, 0)
    states = [B.State(wl.numel, wl.num_workers, wl.momentum, wl.clip_threshold,
                      B.warmup_sparsity(0), sample_ratio=wl.sample_ratio, seed=I.BASE_SEED + w)
              for w in range(NW)]
    pool = [[h.cuda() for h in row] for row in hosts]
    dense = torch.empty(L, dtype=torch.float32, device="cuda")
    weights = torch.randn(L, dtype=torch.float32, device="cuda")
    ws = torch.empty(max(B.decode_workspace_bytes(NW, L), 4), dtype=torch.uint8, device="cuda")
    main_stream = torch.cuda.current_stream()
    NS = max(1, min(args.streams, NW))
    side = [torch.cuda.Stream() for _ in range(NS)] if NS > 1 else [main_stream]
    peak, _ = _peaks()
    rows = []
    it = 0
    for stage in range(5):
        s_ = B.warmup_sparsity(stage)
        for st in states:
            st.set_sparsity(s_)
        nnz = states[0].max_nnz
        out_i = [torch.empty(nnz, dtype=torch.int32, device="cuda") for _ in range(NW)]
        out_v = [torch.empty(nnz, dtype=torch.float32, device="cuda") for _ in range(NW)]

        def step(t):
            if NS > 1:
                ev = torch.cuda.Event()
                ev.record(main_stream)
                for q in side:
                    q.wait_event(ev)
            for w in range(NW):
                states[w].compress(pool[w][t % POOL], out_i[w], out_v[w], stream=side[w % NS])
            if NS > 1:
                for q in side:
                    ev = torch.cuda.Event()
                    ev.record(q)
                    main_stream.wait_event(ev)
            B.decode_accumulate_sgd(out_i, out_v, dense, weights, LR, ws)

        for _ in range(3):
            step(it)
            it += 1
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.stage_iters):
            step(it)
            it += 1
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / args.stage_iters
        nbytes = NW * ((24.0 if wl.clip_threshold > 0 else 20.0) * wl.total + 16.0 * nnz) + \
            4.0 * L + 8.0 * NW * nnz + 12.0 * L
        rows.append({"stage": stage, "sparsity": s_, "nnz_per_worker": nnz, "ms_per_step": ms,
                     "elements_per_s": NW * wl.total / (ms * 1e-3),
                     "algorithmic_gbs": nbytes / (ms * 1e-3) / 1e9,
                     "frac_of_peak": nbytes / (ms * 1e-3) / 1e9 / peak})
    total_ms = sum(r["ms_per_step"] for r in rows) * args.stage_iters
    print(json.dumps({"metric": METRIC, "unit": UNIT, "schedule": "Sec. 4.1 warm-up, 5 stages",
                      "value": NW * wl.total * 5 * args.stage_iters / (total_ms * 1e-3),
                      "config": {"workload": wl.name, "elements": wl.total,
                                 "simulated_workers": NW, "stage_iters": args.stage_iters,
                                 "streams": NS, "clip_threshold": wl.clip_threshold},
                      "stages": rows}))


def run_literal(args):
    """Compress-only timing of the paper-literal sampled selection (select_mode = 1, Sec. 5 as
    stated: variable number of entries, so the fixed-size step of the headline does not apply)."""
    POOL = E2E_POOL
    import torch
    from paper_1712_01887_b200 import build
    build.build()
    from paper_1712_01887_b200 import binding as B
    wl = I.workload(args.workload) if args.workload != "sweep" else I.workload("sweep", n=args.n)
    if args.clip is not None:
        wl.clip_threshold = args.clip
    if args.sparsity is not None:
        wl.sparsity = args.sparsity
    NW = args.workers or wl.num_workers
    off, L, hosts = _make_pool(wl, NW, 0)
    res = {}
    for mode in (0, 1):
        states = [B.State(wl.numel, wl.num_workers, wl.momentum, wl.clip_threshold, wl.sparsity,
                          sample_ratio=wl.sample_ratio, seed=I.BASE_SEED + w, select_mode=mode)
                  for w in range(NW)]
        pool = [[h.cuda() for h in row] for row in hosts]
        cap = states[0].max_nnz
        oi = [torch.empty(cap, dtype=torch.int32, device="cuda") for _ in range(NW)]
        ov = [torch.empty(cap, dtype=torch.float32, device="cuda") for _ in range(NW)]
        for t in range(args.warmup):
            for w in range(NW):
                states[w].compress(pool[w][t % POOL], oi[w], ov[w])
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for t in range(args.steps):
            for w in range(NW):
                states[w].compress(pool[w][t % POOL], oi[w], ov[w])
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / (args.steps * NW)
        total, per = states[0].nnz()
        res["exact" if mode == 0 else "paper_literal"] = {
            "compress_ms": ms, "elements_per_s": wl.total / (ms * 1e-3),
            "entries_sent_last_call": total, "sum_k": int(states[0].k.sum())}
        for st in states:
            st.close()
        del pool
    print(json.dumps({"metric": METRIC, "unit": UNIT, "config": {"workload": wl.name,
                      "elements": wl.total, "sparsity": wl.sparsity, "simulated_workers": NW},
                      "select_modes": res}))


def run_reference(args):
    """--impl reference: the CPU oracle on the same metric and config (bounded sample per step)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = I.workload(args.workload) if args.workload != "sweep" else I.workload("sweep", n=args.n)
    if args.clip is not None:
        wl.clip_threshold = args.clip
    nw = min(2, wl.num_workers)
    step = _oracle_step_factory(wl, nw)
    K, W = args.steps, args.warmup
    for t in range(W):
        step(t)
    t0 = time.perf_counter()
    for t in range(K):
        step(W + t)
    dt = time.perf_counter() - t0
    value = nw * wl.total * K / dt
    sample = (f"each step = {nw} of the {wl.num_workers} simulated workers on the full {wl.name} "
              f"shapes (compress x{nw} + decode + SGD), single thread")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": K, "warmup": W,
        "ms_per_step": dt / K * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": wl.name, "tensors": len(wl.shapes), "elements": wl.total,
                   "simulated_workers": nw, "sparsity": wl.sparsity, "momentum": wl.momentum,
                   "clip_threshold": wl.clip_threshold,
                   "sample": f"{nw} of the workload's {wl.num_workers} simulated workers per "
                             "step (a bounded sample: the metric is per element, the decode "
                             f"sums {nw} lists instead of {wl.num_workers})"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle",
                         "sample": sample, "host_cpus": os.cpu_count()},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="resnet50",
                    choices=["cfg1", "resnet50", "lstm", "lstm_small", "deepspeech",
                             "deepspeech_small", "sweep"])
    ap.add_argument("--n", type=int, default=1 << 24, help="tensor length for --workload sweep")
    ap.add_argument("--workers", type=int, default=None, help="simulated workers (default: config)")
    ap.add_argument("--clip", type=float, default=None, help="override thr_G (0 = off)")
    ap.add_argument("--sparsity", type=float, default=None)
    ap.add_argument("--streams", type=int, default=8, help="streams the workers' compress calls use")
    ap.add_argument("--no-batch", action="store_true",
                    help="one dgc_compress per worker on --streams streams instead of "
                         "dgc_compress_batch")
    ap.add_argument("--flush-l2", action="store_true",
                    help="rewrite a 256 MB buffer before every timed step (cold L2) and sum "
                         "per-step event times")
    ap.add_argument("--timeline", action="store_true",
                    help="add the GPU-clock timeline of one step (per worker and kernel: first "
                         "and last block start) to the JSON line")
    ap.add_argument("--graph", action="store_true",
                    help="capture the step into CUDA graphs (one per pooled gradient) and time "
                         "their replays")
    ap.add_argument("--separate-receive", action="store_true",
                    help="decode and SGD as two calls instead of the one-pass entry point")
    ap.add_argument("--repeats", type=int, default=3,
                    help="times the timed region of exactly --steps steps is run; the median "
                         "is reported, all of them listed")
    ap.add_argument("--pool", type=int, default=None,
                    help="distinct gradients per worker (default: the workload's iteration "
                         "count, at most 10)")
    ap.add_argument("--no-second", action="store_true",
                    help="skip the second target workload (LSTM-shaped set) of the default run")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    ap.add_argument("--compare-select-modes", action="store_true",
                    help="compress-only timing of exact vs paper-literal sampled selection")
    ap.add_argument("--warmup-schedule", action="store_true",
                    help="run the 5-stage sparsity warm-up and report per-stage timings")
    ap.add_argument("--stage-iters", type=int, default=20)
    ap.add_argument("--traffic", type=float, default=None,
                    help="DRAM bytes per launch of the dominant kernel from an ncu capture")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    elif args.warmup_schedule:
        run_schedule(args)
    elif args.compare_select_modes:
        run_literal(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

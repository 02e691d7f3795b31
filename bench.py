#!/usr/bin/env python
"""Benchmark of the FlowMM per-layer KV-cache compression on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg5] [--permille 50]
    python bench.py --impl reference ...       # the fp64 CPU oracle as the reference arm

A step is one flowmm_compress_layer call over every (layer, sequence) unit of
the workload's stack (default: the long-context workload cfg5, 80 layers x 4
sequences of 33 792 tokens, the largest one that fits a GPU).  The metric is context tokens compressed per second per
layer: n_seqs * L * n_layers / step time, summed over GPUs (each GPU compresses
its own sequences; units are independent, so there is no collective on the
data path).  Prints one JSON line.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "context tokens compressed/sec per layer (all heads)"
UNIT = "tokens/s/layer"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg5")
    ap.add_argument("--permille", type=int, default=0,
                    help="retention budget in 1/1000 of the context (0: 100 if the workload lists it, else its first)")
    ap.add_argument("--layers", type=int, default=0, help="use only the first N layers (0 = the whole stack)")
    ap.add_argument("--path", default="auto", choices=["auto", "simt"])
    ap.add_argument("--sets", type=int, default=0, help="rotating input sets held on the device (0 = automatic)")
    ap.add_argument("--launch", choices=["graph", "plain"], default="plain",
                    help="plain: the timed steps are the library calls (default); graph: the steps are also replayed "
                         "from CUDA graphs captured from the call and that time is reported beside the value")
    ap.add_argument("--cpu-seconds", type=float, default=20.0, help="CPU time the oracle baseline leg may spend")
    ap.add_argument("--reference-seconds", type=float, default=150.0,
                    help="--impl reference: wall time its warm-up and timed steps may spend together")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-decode", action="store_true", help="skip the decode-attention timing over the caches")
    ap.add_argument("--no-e2e", action="store_true", help="skip the end-to-end leg (host buffers), e.g. under a profiler")
    ap.add_argument("--cpu-baseline-units", type=int, default=0)
    return ap.parse_args()


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """SM clock and throttle-reason samples taken through NVML while the timed region runs
    (read-only queries, a few milliseconds apart, from a helper thread)."""

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.samples, self.reasons = [], set()
        self.sm_max = None
        self._stop = False
        self._thread = None
        self._err = None
        self._ready = None
        self._mark = 0

    def _run(self):
        try:
            import pynvml as nv
            nv.nvmlInit()
            vis = os.environ.get("CUDA_VISIBLE_DEVICES")
            idx = self.gpu
            if vis:
                ids = [x for x in vis.split(",") if x.strip() != ""]
                if self.gpu < len(ids) and ids[self.gpu].strip().isdigit():
                    idx = int(ids[self.gpu])
            h = nv.nvmlDeviceGetHandleByIndex(idx)
            self.sm_max = float(nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM))
            get_reasons = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
                nv.nvmlDeviceGetCurrentClocksThrottleReasons
            table = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}
            while not self._stop:
                self.samples.append(float(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM)))
                bits = int(get_reasons(h))
                for bit, name in table.items():
                    if bits & bit:
                        self.reasons.add(name)
                self._ready.set()
                time.sleep(0.002)
        except Exception as exc:            # NVML missing or refused: report it, do not fail the run
            self._err = repr(exc)
            self._ready.set()

    def start(self):
        """Starts the helper thread and returns once its first sample is in (NVML is up by then)."""
        import threading
        self._ready = threading.Event()
        self._thread = threading.Thread(target=self._run, daemon=True)
        self._thread.start()
        self._ready.wait(timeout=30)

    def mark(self):
        """Samples taken before this call (warm-up, idle) are left out of the summary."""
        self._mark = len(self.samples)
        self.reasons.clear()

    def stop(self):
        self._stop = True
        if self._thread is not None:
            self._thread.join(timeout=5)
        timed = self.samples[self._mark:]
        out = {"sm_mhz": statistics.median(timed) if timed else None, "sm_max_mhz": self.sm_max,
               "samples": len(timed), "reasons": sorted(self.reasons)}
        if self._err:
            out["error"] = self._err
        return out


def match_pair_count(p, tau_eff, diag, modality):
    """Number of (non-pivot, admissible pivot) pairs whose similarity Eq. 9-10 need, summed over
    all units and heads: the gate of Eq. 10 removes pivots above tau, an intra-modal layer pairs
    tokens of equal modality only.  Counted from one call's own outputs; accounting only."""
    import torch
    imp, ret, strat = diag["importance"], diag["retained"].long(), diag["strategy"]
    U, Hkv, L = imp.shape
    mod = modality.bool()[:, None, :].expand(U, Hkv, L)
    adm = torch.gather(imp, 2, ret) <= tau_eff
    ret_vis = torch.gather(mod, 2, ret)
    n_v = (adm & ret_vis).sum(-1).double()
    n_t = (adm & ~ret_vis).sum(-1).double()
    tot_vis = modality.bool().sum(-1).double()[:, None]
    e_v = tot_vis - ret_vis.sum(-1).double()
    e_t = (L - tot_vis) - (~ret_vis).sum(-1).double()
    cross = (strat == 1).double()[:, None]
    pairs = cross * (e_t + e_v) * (n_t + n_v) + (1 - cross) * (e_t * n_t + e_v * n_v)
    return float(pairs.sum().item())


def kernel_model(wl, B, dsize):
    """Algorithmic flops and bytes of each kernel for ONE unit (all heads), from the
    operation's definition: what must be read and written once, and the multiply-adds of the
    two contractions."""
    Hq, Hkv, L, W, D = wl.n_q_heads, wl.n_kv_heads, wl.seq_len, wl.window, wl.head_dim
    E = L - B
    score_flops = 2.0 * Hq * W * L * D
    score_bytes = (Hkv * L * D + Hq * W * D) * dsize
    m = {
        "score_stats": (score_flops, score_bytes),
        "score_colsum": (score_flops, score_bytes + 4.0 * Hkv * L),
        "inv_norm": (2.0 * Hkv * L * D, Hkv * L * D * dsize + 4.0 * Hkv * L),
        "match": (2.0 * Hkv * E * B * D, Hkv * L * D * dsize + 8.0 * Hkv * E),
        "merge_pieces": (4.0 * Hkv * L * D, 2.0 * Hkv * (L + B) * D * dsize),
        "select_topb": (0.0, 4.0 * Hkv * L * 2),
        "build_csr": (0.0, 4.0 * Hkv * E * 3),
    }
    return m


def csrc_digest():
    """sha256 over the CUDA sources and the public header, in name order: identifies the kernels as built."""
    import hashlib
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2511_05534_b200", "csrc")
    for path in sorted(os.path.join(csrc, f) for f in os.listdir(csrc)) + [os.path.join(ROOT, "include", "flowmm.h")]:
        h.update(os.path.basename(path).encode())
        h.update(open(path, "rb").read())
    return h.hexdigest()[:16]


def ncu_traffic(workload, permille, units, kernel):
    """DRAM bytes (read + write) of one launch of `kernel` from the committed table of ncu captures
    (paper_2511_05534_b200/ncu_traffic.json; the summaries under profiles/ give the commands).  An entry is
    per unit of its workload and budget, taken on a small case, and scaled by the units of this call (traffic
    of these kernels grows in proportion to the units).  None when there is no entry, or when the sources have
    changed since the counters were taken."""
    path = os.path.join(ROOT, "paper_2511_05534_b200", "ncu_traffic.json")
    if not os.path.exists(path):
        return None
    table = json.load(open(path))
    if table.get("csrc_digest") != csrc_digest():
        return None
    per_unit = table.get("bytes_per_unit", {}).get("%s@%d" % (workload, permille), {}).get(kernel)
    return None if per_unit is None else per_unit * units


KERNEL_MODEL = {   # kernel name -> entry of kernel_model()
    "score_stats_simt": "score_stats", "score_stats_tc": "score_stats", "score_fused_tc": "score_colsum",
    "score_colsum_simt": "score_colsum", "score_colsum_tc": "score_colsum",
    "inv_norm": "inv_norm", "match_simt": "match", "match_tc": "match", "match_small_tc": "match", "merge_pieces": "merge_pieces",
    "merge_tc": "merge_pieces", "merge_staged": "merge_pieces",
    "select_topb": "select_topb", "build_csr": "build_csr",
}


# Share of a scoring kernel's exponentials that it evaluates as a polynomial on the FMA pipe (the kernels' own
# constants: score_tc.cuh); the rest goes through the exp2 unit.
EXP_FMA_SHARE = {"score_stats_tc": 0.25, "score_colsum_tc": 0.25}


def model_for(name, model):
    return model.get(KERNEL_MODEL.get(name, ""), (0.0, 0.0))


def _oracle_sample(wl, permille, n_units):
    """A bounded sample of the workload for the oracle: `n_units` layers spread over the stack, sequence 0."""
    from oracle import flowmm_oracle as O
    from paper_2511_05534_b200 import inputs
    B = wl.n_keep(permille)
    n_units = max(1, min(n_units, wl.n_layers))
    layers = sorted(set(int(round(i * (wl.n_layers - 1) / max(1, n_units - 1))) for i in range(n_units)))
    if n_units == 1:
        layers = [wl.n_layers // 2]
    units = [(l, 0) for l in layers]
    data = inputs.make_units(wl, units)
    p = O.OracleParams(len(units), wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.seq_len, wl.window, B,
                       theta=wl.theta, tau=wl.tau_rel, tau_mode=O.TAU_REL)
    return p, data, layers


def _oracle_units_per_step(wl):
    """How many layers of the stack one oracle step covers, by context length (a step of seconds, not minutes)."""
    return 8 if wl.seq_len <= 1024 else (4 if wl.seq_len <= 4096 else (2 if wl.seq_len <= 16384 else 1))


def run_reference(args):
    """The oracle as the reference arm: each step compresses a bounded sample of the stack; warm-up and timed
    steps together are held to --reference-seconds of wall time (fewer steps are timed if they would not fit,
    and the line says how many were)."""
    from oracle import flowmm_oracle as O
    from paper_2511_05534_b200 import configs

    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = configs.get(args.workload)
    B = wl.n_keep(args.permille)
    O.build()
    p, data, layers = _oracle_sample(wl, args.permille, _oracle_units_per_step(wl))

    def one():
        t0 = time.perf_counter()
        O.compress_layer(p, data["q"], data["k"], data["v"], data["modality"])
        return time.perf_counter() - t0

    budget = max(1.0, args.reference_seconds)
    spent, warm = 0.0, 0
    while warm < max(1, args.warmup) and (warm == 0 or spent + spent / warm <= 0.2 * budget):
        spent += one()
        warm += 1
    per_step = spent / warm
    steps = max(1, min(max(1, args.steps), int((budget - spent) / per_step)))
    times = [one() for _ in range(steps)]
    dt = sum(times) / steps
    value = wl.seq_len * len(layers) / dt
    sample = ("layers %s of the %s stack, one sequence, per step; %d warm-up and %d timed steps (asked: %d and %d; "
              "held to %.0f s of wall time)" % (layers, wl.name, warm, steps, args.warmup, args.steps, budget))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
        "warmup": warm, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "layers": wl.n_layers, "seqs": wl.n_seqs, "budget_permille": args.permille,
                   "n_keep": B, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": O.threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def cpu_baseline(wl, permille, n_units, seconds):
    """The oracle as it stands on the host cores, on a bounded sample: repeated until `seconds` of CPU wall
    time are spent (at least once, at most 20 times)."""
    from oracle import flowmm_oracle as O

    if n_units <= 0:
        n_units = wl.n_layers if wl.seq_len <= 1024 else _oracle_units_per_step(wl)
    O.build()
    p, data, layers = _oracle_sample(wl, permille, n_units)
    reps, t_total = 0, 0.0
    while reps < 20 and (reps == 0 or t_total + t_total / reps <= seconds):
        t0 = time.perf_counter()
        O.compress_layer(p, data["q"], data["k"], data["v"], data["modality"])
        t_total += time.perf_counter() - t0
        reps += 1
    dt = t_total / reps
    return {"value": wl.seq_len * len(layers) / dt, "unit": UNIT, "cores": O.threads(), "kind": "oracle",
            "sample": "%d layer(s) %s of the %d-layer %s stack, one of its %d sequence(s), %d repetition(s), %.1f s of CPU "
                      "wall time" % (len(layers), layers, wl.n_layers, wl.name, wl.n_seqs, reps, t_total)}


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2511_05534_b200 import binding as F
    from paper_2511_05534_b200 import build, configs, inputs, shard

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    build.build()
    F.load()

    wl = configs.get(args.workload)
    n_layers = args.layers if args.layers > 0 else wl.n_layers
    units = shard.rank_units(n_layers, wl.n_seqs, rank, world)
    U = len(units)
    B = wl.n_keep(args.permille)
    dt_code = F.BF16 if wl.dtype == "bf16" else F.F32
    dsize = 2 if wl.dtype == "bf16" else 4
    p = F.Params(U, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.seq_len, wl.window, B, dtype=dt_code,
                 theta=wl.theta, tau=wl.tau_rel, tau_mode=F.TAU_REL,
                 path=F.PATH_SIMT if args.path == "simt" else F.PATH_AUTO)

    # several independent input sets, rotated, so that a step never finds its inputs in L2
    bytes_per_set = 2 * U * wl.n_kv_heads * wl.seq_len * wl.head_dim * dsize
    n_sets = max(2, min(8, int(1.5e9 // max(1, bytes_per_set)) + 1))
    if bytes_per_set > 20e9:
        n_sets = 1            # a set this large cannot stay in the 126 MB L2 anyway
    if args.sets > 0:
        n_sets = args.sets
    sets = [inputs.make_stack_device(wl, dev, units, seed_offset=shard.seed_offset(rank, i)) for i in range(n_sets)]
    k_out = torch.empty((U, wl.n_kv_heads, B, wl.head_dim), dtype=sets[0][1].dtype, device=dev)
    v_out = torch.empty_like(k_out)
    ws = F.alloc_workspace(p, dev)

    def step(i):
        q, k, v, m = sets[i % n_sets]
        F.flowmm_compress_layer(p, q, k, v, m, k_out, v_out, ws)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()                          # returns after its first sample: NVML is up before anything is timed
    for i in range(max(3, args.warmup)):
        step(i)
    launches_per_step = F.flowmm_last_launch_count()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # the timed region: exactly --steps plain library calls, CUDA events on the launching stream
    sampler.mark()
    e0.record()
    for i in range(args.steps):
        step(i)
    e1.record()
    barrier()
    ms_total = e0.elapsed_time(e1)
    clocks = sampler.stop() if rank == 0 else None
    status = F.flowmm_last_device_status(ws)
    if status != 0:
        raise RuntimeError("device status: " + F.status_string(status))
    # Beside it, on request: the same steps replayed from CUDA graphs captured from the call, one per input set
    # (the call is stream-ordered and allocation-free; same kernels and work, only the host's launch gaps go).
    graph_ms_step = None
    if args.launch == "graph":
        try:
            graphs, side = [], torch.cuda.Stream(device=dev)
            with torch.cuda.stream(side):
                step(0)                          # (function attributes, symbol look-ups) on the capturing stream
                torch.cuda.synchronize()
                for i in range(n_sets):
                    g = torch.cuda.CUDAGraph()
                    # (thread_local: calls of other threads, a process group's watchdog for one, do not disturb the capture)
                    with torch.cuda.graph(g, stream=side, capture_error_mode="thread_local"):
                        step(i)
                    graphs.append(g)
            torch.cuda.synchronize()
            for i in range(3):
                graphs[i % n_sets].replay()
            barrier()
            e0.record()
            for i in range(args.steps):
                graphs[i % n_sets].replay()
            e1.record()
            barrier()
            graph_ms_step = shard.max_over_ranks(e0.elapsed_time(e1), dev) / args.steps
            del graphs
        except Exception as exc:                 # capture refused: say so, the plain timing stands
            sys.stderr.write("graph capture failed (%s)\n" % exc)
    ms_total = shard.max_over_ranks(ms_total, dev)
    ms_step = ms_total / args.steps
    tokens_layers = wl.n_seqs * wl.seq_len * n_layers        # tokens x layers compressed per step per GPU
    value = shard.aggregate_throughput(tokens_layers, world, ms_step)

    # per-kernel attribution: the same steps again with an event after every kernel
    F.flowmm_profile_enable(True)
    per_kernel = {}
    for i in range(args.steps):
        step(i)
        for name, ms in F.flowmm_profile_read():
            per_kernel.setdefault(name, []).append(ms)
    F.flowmm_profile_enable(False)
    torch.cuda.synchronize()
    peaks = load_peaks()
    model = kernel_model(wl, B, dsize)
    # the match step's own flops: only pairs that pass the gates of Eq. 10 need a similarity
    tau_eff = wl.tau_rel * wl.window / wl.seq_len
    q0, k0, v0, m0 = sets[0]
    diag = F.compress_layer_alloc(p, q0, k0, v0, m0, ws=ws)
    pairs = match_pair_count(p, tau_eff, diag, m0)
    dense_pairs = float(U) * wl.n_kv_heads * (wl.seq_len - B) * B
    del diag
    # Three ceilings per kernel: the tensor cores (sustained bf16 peak), HBM, and for the scoring passes the
    # exp2 unit: one exponential per attention logit and pass, 16 results per clock per SM, at the SM clock
    # sampled during the timed region, less the share of exponentials the kernel evaluates as a polynomial on
    # the FMA pipe instead (EXP_FMA_SHARE).  A kernel is measured against the slowest of its ceilings.
    sm_mhz = (clocks or {}).get("sm_mhz") or (clocks or {}).get("sm_max_mhz") or 1965.0
    exp_peak = 16.0 * torch.cuda.get_device_properties(dev).multi_processor_count * sm_mhz * 1e6   # exponentials / s
    n_exp_unit = float(wl.n_q_heads) * wl.window * wl.seq_len
    kernels = {}
    for name, times in per_kernel.items():
        avg = sum(times) / len(times)
        flops, nbytes = model_for(name, model)
        flops, nbytes = flops * U, nbytes * U
        if KERNEL_MODEL.get(name) == "match":
            flops = 2.0 * wl.head_dim * pairs
        n_exp = n_exp_unit * U * (1.0 - EXP_FMA_SHARE[name]) if name in EXP_FMA_SHARE else 0.0
        t = {"tensor": flops / (peaks["bf16_tflops_sustained"] * 1e12) if dt_code == F.BF16 else 0.0,
             "hbm": nbytes / (peaks["hbm_gbs"] * 1e9), "alu": n_exp / exp_peak}
        bound = max(t, key=lambda b: t[b])
        kernels[name] = {"ms": avg, "bound": bound, "gbs": nbytes / (avg * 1e-3) / 1e9,
                         "tflops": flops / (avg * 1e-3) / 1e12, "frac": t[bound] / (avg * 1e-3)}
        if n_exp > 0:
            kernels[name].update({"gexp_s": n_exp / (avg * 1e-3) / 1e9, "frac_tensor": t["tensor"] / (avg * 1e-3),
                                  "frac_exp_unit": t["alu"] / (avg * 1e-3)})
    top = max(kernels, key=lambda n: kernels[n]["ms"])
    tk = kernels[top]
    if tk["bound"] == "tensor":
        roofline = {"kernel": top, "bound": "tensor", "achieved": tk["tflops"], "peak": peaks["bf16_tflops_sustained"],
                    "unit": "TFLOP/s", "frac": tk["frac"], "traffic": None,
                    "peak_source": peaks["source"] + " (sustained bf16)"}
    elif tk["bound"] == "alu":
        roofline = {"kernel": top, "bound": "alu", "achieved": tk["gexp_s"], "peak": exp_peak / 1e9,
                    "unit": "Gexp2/s", "frac": tk["frac"], "traffic": None, "frac_tensor": tk["frac_tensor"],
                    "peak_source": "derived: 16 exp2 per clock per SM x %d SMs x %.0f MHz sampled; exponentials the "
                                   "kernel sends to the FMA pipe (%.0f %%) are not counted" %
                                   (torch.cuda.get_device_properties(dev).multi_processor_count, sm_mhz,
                                    100 * EXP_FMA_SHARE[top])}
    else:
        roofline = {"kernel": top, "bound": "hbm", "achieved": tk["gbs"], "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": tk["frac"], "traffic": None, "peak_source": peaks["source"]}
    roofline["launch_ms"] = tk["ms"]
    roofline["traffic"] = ncu_traffic(wl.name, args.permille, U, top)
    roofline["traffic_unit"] = "bytes per launch (ncu dram__bytes_read.sum + dram__bytes_write.sum, scaled from a small capture by units)"
    roofline["algorithmic_bytes"] = model_for(top, model)[1] * U
    roofline["share_of_step"] = tk["ms"] / sum(k2["ms"] for k2 in kernels.values())

    # end to end: pinned host inputs -> device -> compress -> pinned host result, every step.  Two streams with their
    # own device buffers take the steps alternately, so that one step's result goes back to the host while the next
    # step's inputs come in (the two directions of the host link); every step still moves all of its bytes.
    def end_to_end():
        # every rank of the node pins a whole input set: all ranks agree beforehand on whether the host has room
        import psutil
        need = sum(t.numel() * t.element_size() for t in sets[0]) + 2 * k_out.numel() * k_out.element_size()
        fits = torch.tensor([1.0 if psutil.virtual_memory().available > 1.2 * need * world else 0.0], device=dev)
        if world > 1:
            dist.all_reduce(fits, op=dist.ReduceOp.MIN)
        if fits.item() == 0.0:
            raise MemoryError("host memory cannot hold %d pinned input sets of %.1f GB" % (world, need / 1e9))
        hq, hk, hv, hm = (t.cpu().pin_memory() for t in sets[0])
        h2d = sum(t.numel() * t.element_size() for t in (hq, hk, hv, hm))
        lanes = []
        for _ in range(2 if bytes_per_set < 8e9 else 1):
            lanes.append({"s": torch.cuda.Stream(device=dev), "in": [torch.empty_like(t) for t in sets[0]],
                          "ko": torch.empty_like(k_out), "vo": torch.empty_like(v_out), "ws": F.alloc_workspace(p, dev),
                          "hko": torch.empty_like(k_out, device="cpu").pin_memory(),
                          "hvo": torch.empty_like(v_out, device="cpu").pin_memory()})
        d2h = sum(t.numel() * t.element_size() for t in (lanes[0]["hko"], lanes[0]["hvo"]))
        e2e_steps = max(4, min(args.steps, 10))

        def e2e_step(i):
            ln = lanes[i % len(lanes)]
            with torch.cuda.stream(ln["s"]):
                for d, h in zip(ln["in"], (hq, hk, hv, hm)):
                    d.copy_(h, non_blocking=True)
                F.flowmm_compress_layer(p, *ln["in"], ln["ko"], ln["vo"], ln["ws"])
                ln["hko"].copy_(ln["ko"], non_blocking=True)
                ln["hvo"].copy_(ln["vo"], non_blocking=True)

        for i in range(len(lanes)):
            e2e_step(i)
        barrier()
        t_host0 = time.perf_counter()
        for ln in lanes:
            ln["s"].wait_stream(torch.cuda.current_stream())
        e0.record()
        for ln in lanes:
            ln["s"].wait_event(e0)
        for i in range(e2e_steps):
            e2e_step(i)
        for ln in lanes:
            torch.cuda.current_stream().wait_stream(ln["s"])
        e1.record()
        barrier()
        e2e_ms = e0.elapsed_time(e1)
        e2e_wall_ms = (time.perf_counter() - t_host0) * 1e3
        for ln in lanes:
            status = F.flowmm_last_device_status(ln["ws"])
            if status != 0:
                raise RuntimeError("device status (end to end): " + F.status_string(status))
        e2e_ms = shard.max_over_ranks(e2e_ms, dev)
        e2e_value = shard.aggregate_throughput(tokens_layers, world, e2e_ms / e2e_steps)
        del lanes
        return {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": e2e_steps, "wall_ms_per_step": round(e2e_wall_ms / e2e_steps, 4)}


    try:
        e2e = {"value": None, "unit": UNIT, "skipped": "--no-e2e"} if args.no_e2e else end_to_end()
    except (RuntimeError, MemoryError) as exc:      # e.g. the host cannot pin a whole input set: say so, keep the line
        if "device status" in str(exc):
            raise
        e2e = {"value": None, "unit": UNIT, "h2d_bytes_per_step": None, "d2h_bytes_per_step": None,
               "error": str(exc).splitlines()[0][:200]}
    torch.cuda.synchronize()

    # the step this path feeds (not part of the timed metric): one decode query per head over every layer's
    # cache, full length against compressed; L2 flushed before every call, each call timed on its own
    decode = None
    if not args.no_decode:
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
        comp = []
        for q, k, v, m in sets:
            ko, vo = torch.empty_like(k_out), torch.empty_like(v_out)
            F.flowmm_compress_layer(p, q, k, v, m, ko, vo, ws)
            comp.append((ko, vo))
        q_dec = [t[0][:, :, -1, :].contiguous() for t in sets]
        out_dec = torch.empty(q_dec[0].shape, dtype=torch.float32, device=dev)
        decode = {}
        for label, caches in (("full", [(t[1], t[2]) for t in sets]), ("compressed", comp)):
            ws_d = torch.empty(F.flowmm_decode_workspace_bytes(q_dec[0], *caches[0]), dtype=torch.uint8, device=dev)
            times = []
            for i in range(3 + 10):
                kk, vv = caches[i % n_sets]
                flush.zero_()
                e0.record()
                F.flowmm_decode_attention(q_dec[i % n_sets], kk, vv, out_dec, ws_d)
                e1.record()
                torch.cuda.synchronize()
                if i >= 3:
                    times.append(e0.elapsed_time(e1))
            status = F.flowmm_last_device_status(ws_d)
            if status != 0:
                raise RuntimeError("device status (decode): " + F.status_string(status))
            ms = sorted(times)[len(times) // 2]
            nbytes = 2 * caches[0][0].numel() * dsize
            decode[label] = {"n_keys": caches[0][0].shape[2], "ms": round(ms, 5), "bytes": nbytes,
                             "gbs": round(nbytes / (ms * 1e-3) / 1e9, 1),
                             "frac_hbm": round(nbytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"], 4)}
        decode["speedup"] = round(decode["full"]["ms"] / decode["compressed"]["ms"], 3)
        decode["what"] = "flowmm_decode_attention, one query per head, all %d units in one call, per GPU" % U
        del comp, flush

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": wl.dtype, "data": "synthetic",
            "config": {"workload": wl.name, "layers": n_layers, "seqs": wl.n_seqs, "n_q_heads": wl.n_q_heads,
                       "n_kv_heads": wl.n_kv_heads, "head_dim": wl.head_dim, "seq_len": wl.seq_len,
                       "window": wl.window, "budget_permille": args.permille, "n_keep": B,
                       "units_per_call": U, "match_pairs_fraction_of_dense": round(pairs / max(1.0, dense_pairs), 4),
                       "launch": "plain flowmm_compress_layer calls",
                       "l2": "%d rotating input sets of %.0f MB (inputs larger than L2)" %
                       (n_sets, bytes_per_set / 1e6), "path": args.path, "parallelism": "units sharded, no collective"},
            "clocks": clocks,
            "e2e": e2e,
            "gpu_launches": launches_per_step * args.steps,
            "roofline": roofline,
            "kernels": {n: {k2: (round(v2, 5) if isinstance(v2, float) else v2) for k2, v2 in d.items()}
                        for n, d in kernels.items()},
        }
        if graph_ms_step is not None:
            line["graph_replay_ms_per_step"] = graph_ms_step
        if decode is not None:
            line["decode"] = decode
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(wl, args.permille, args.cpu_baseline_units, args.cpu_seconds)
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    args = parse_args()
    if args.permille <= 0:
        from paper_2511_05534_b200 import configs
        budgets = configs.get(args.workload).budgets_permille
        args.permille = 100 if 100 in budgets else budgets[0]
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

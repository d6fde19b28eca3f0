#!/usr/bin/env python
"""Benchmark of the hybrid-attention forward pass (one layer = one step).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload wan81]

Prints ONE JSON line.  A step is one pass of the whole hot path (K pass -> state reduction ->
Q pass) over one synthetic layer input already resident in HBM; `e2e` is the same step through
the host-buffer entry point with the host<->device copies inside the timed region.  With
N > 1 (torchrun) every rank runs its own layer input (independent batches, no collective in
the data path) and the value is the aggregate over ranks.  `--impl reference` times the
float64 CPU oracle on the host cores instead (a deliberately slow baseline).
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "hybrid-attn fwd tokens/s per layer at N=32760 (12x128 heads); % of bf16 tensor peak"

KERNEL_SOURCES = ("tensor_qpass.cu", "tensor_qstream.cu", "tensor_kpass.cu", "tensor_common.cuh", "sm100_ptx.cuh", "sm100_tmem_wide.cuh")


def kernel_source_digest(names=KERNEL_SOURCES):
    """sha256 over the source files a kernel is built from (the ncu summaries record it at capture time)."""
    import hashlib
    h = hashlib.sha256()
    for n in names:
        with open(os.path.join(ROOT, "paper_2509_24899_b200", "csrc", n), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def measured_dram_traffic(kernel, workload):
    """DRAM bytes of one launch (dram__bytes_read.sum + dram__bytes_write.sum) from the committed ncu summary
    profiles/<kernel>_<workload>.txt, or None when there is no summary or the kernel's sources have changed
    since the capture (the summary carries the digest of the sources it was taken with)."""
    path = os.path.join(ROOT, "profiles", "%s_%s.txt" % (kernel, workload))
    if not os.path.exists(path):
        return None
    fields = {}
    with open(path) as f:
        for line in f:
            if ":" in line:
                k, v = line.split(":", 1)
                fields[k.strip()] = v.strip()
    try:
        if fields["source_digest"] != kernel_source_digest():
            return None
        return int(fields["dram_bytes_read_per_launch"]) + int(fields["dram_bytes_write_per_launch"])
    except (KeyError, ValueError):
        return None


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained"), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def flops_per_layer(wl, n_s):
    """Algorithmic FLOPs of one layer (all heads), split per kernel.  Per token the feature map costs
    2 d F (one layer) or 2 d hidden + 2 hidden F (two layers); state and apply cost 2 F (d + 1) each."""
    N, d, F = wl.N, wl.d, wl.F
    n_l = N - n_s
    heads = wl.B * wl.H
    phi = 2 * d * F if wl.layers == 1 else 2 * d * wl.hidden_width + 2 * wl.hidden_width * F
    kpass = (phi * n_l + 2 * n_l * F * (d + 1)) if n_l > 0 else 0
    qpass = 4 * N * n_s * d + ((N * phi + 2 * N * F * (d + 1)) if n_l > 0 else 0)
    return {"kpass": heads * kpass, "qpass": heads * qpass, "total": heads * (kpass + qpass)}


def bytes_per_layer(wl):
    """Algorithmic HBM bytes of one layer: q, k, v read once, out written once."""
    return 4 * wl.B * wl.H * wl.N * wl.d * 2


def config_of(wl, n_softmax, world):
    """The `config` object of the JSON line: the workload, named the same way by both arms."""
    return {"workload": wl.name, "B": wl.B, "H": wl.H, "N": wl.N, "d": wl.d, "F": wl.F, "rate": wl.rate,
            "n_softmax": int(n_softmax), "stab_mode": "paper",
            "phi": "%d layer(s), hidden %d, F %d, degree %d" % (wl.layers, wl.hidden_width if wl.layers == 2 else 0, wl.F, wl.degree),
            "parallelism": "dp%d (independent layer inputs per rank)" % world}


def rank_workload(wl, rank):
    """Every rank draws its own layer input (independent batches: weak scaling, no exchange step)."""
    import dataclasses
    return dataclasses.replace(wl, seed=wl.seed + rank)


def max_over_ranks(values, device):
    """Element-wise maximum of a list of per-rank numbers over all ranks (identity without a process group)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def whole_job_value(wl, world, steps, ms):
    """Tokens per second of the whole job: every rank processed `steps` layers of B*N tokens in `ms`."""
    return wl.B * wl.N * world * steps / (ms * 1e-3)


class ClockSampler:
    """Samples SM clock and clock-event reasons of one GPU through NVML in a background thread."""

    def __init__(self, index: int, period_s: float = 0.02):
        self.period, self.samples, self._stop = period_s, [], threading.Event()
        self.max_mhz, self.ok = None, False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            idx = index
            vis = os.environ.get("CUDA_VISIBLE_DEVICES")
            if vis:
                try:
                    idx = int(vis.split(",")[index])
                except ValueError:
                    idx = index
            self.h = pynvml.nvmlDeviceGetHandleByIndex(idx)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False
        self.thread = threading.Thread(target=self._run, daemon=True)

    def _run(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                mhz = nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)
                try:
                    reasons = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    reasons = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                self.samples.append((mhz, reasons))
            except Exception:
                pass
            time.sleep(self.period)

    def start(self):
        if self.ok:
            self.thread.start()

    def reset(self):
        self.samples = []

    def stop(self):
        self._stop.set()
        if self.ok and self.thread.is_alive():
            self.thread.join(timeout=1.0)

    def summary(self):
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["unavailable"], "samples": 0}
        bits = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
                0x4: "sw_power_cap", 0x80: "hw_power_brake_slowdown", 0x10: "sync_boost"}
        seen = set()
        for _, r in self.samples:
            for b, name in bits.items():
                if r & b:
                    seen.add(name)
        return {"sm_mhz": statistics.median(m for m, _ in self.samples), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(seen), "samples": len(self.samples)}


def head_weights(data64, which, h):
    """One head's feature map in the form the oracle takes: a matrix, or a list of layers, each a matrix or a
    (matrix, bias) pair (argument marshalling only)."""
    def layer(wname, bname):
        return (data64[wname][h], data64[bname][h]) if bname in data64 else data64[wname][h]
    first = layer("w" + which, "b" + which + "1")
    if ("w" + which + "2") not in data64:
        return first if not isinstance(first, tuple) else [first]
    return [first, layer("w" + which + "2", "b" + which + "2")]


def cpu_oracle_rate(wl, data64, mask, budget_s, heads=1, rows0=256):
    """Times the float64 oracle on a bounded sample and extrapolates to tokens/s of a full layer.

    Sample: `heads` heads; the linear state over all tokens (timed alone), then the full operator on
    `rows` query rows.  Per-row cost = (t_rows - t_state) / rows; a full layer costs
    H * (t_state + N * t_row) per batch element."""
    from oracle import hybrid_attention as O
    import numpy as np
    n_l = int((~mask).sum())
    q, k, v = data64["q"][0], data64["k"][0], data64["v"][0]

    def one(rows):
        t_state = t_rows = 0.0
        for h in range(heads):
            if n_l > 0:
                t0 = time.perf_counter()
                O.linear_state(k[h], v[h], head_weights(data64, "k", h), mask, wl.degree)
                t_state += time.perf_counter() - t0
            t0 = time.perf_counter()
            O.hybrid_attention_head(q[h], k[h], v[h], head_weights(data64, "q", h), head_weights(data64, "k", h), mask,
                                    None, O.STAB_PAPER, wl.degree, rows=rows)
            t_rows += time.perf_counter() - t0
        return t_state / heads, t_rows / heads

    rows = np.arange(min(rows0, wl.N))
    ts, tr = one(rows)
    t_row = max(tr - ts, 1e-9) / len(rows)
    # grow the sample towards the budget
    want = int(min(wl.N, max(len(rows), (budget_s / heads - 2 * ts) / t_row)))
    if want > 2 * len(rows):
        rows = np.arange(want)
        ts, tr = one(rows)
        t_row = max(tr - ts, 1e-9) / len(rows)
    layer_s = wl.H * (ts + wl.N * t_row)            # per batch element
    return {"tokens_per_s": wl.N / layer_s, "rows": int(len(rows)), "heads": heads,
            "t_state_s": ts, "t_rows_s": tr, "step_s": heads * (ts + tr)}


def run_reference(args, wl):
    """The oracle, as it stands, on the host cores: K timed steps of a bounded sample each."""
    import numpy as np
    from oracle import hybrid_attention as O
    from paper_2509_24899_b200 import workloads as W
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    cores = os.cpu_count() or 1
    data64 = {k: W.bf16_bits_to_f64(v) for k, v in W.generate(wl, heads=1).items()}
    mask = O.softmax_token_mask(wl.grid, wl.block, wl.rate)
    total = args.steps + args.warmup
    budget = max(0.05, min(2.0, 150.0 / total))
    vals, step_s, last = [], [], None
    for i in range(total):
        r = cpu_oracle_rate(wl, data64, mask, budget_s=budget, heads=1, rows0=128)
        if i >= args.warmup:
            vals.append(r["tokens_per_s"])
            step_s.append(r["step_s"])
            last = r
    value = statistics.mean(vals)                      # one host, whatever N is
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * wl.B * wl.N / value,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_of(wl, mask.sum(), args.gpus),
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle",
                         "sample": "per step: 1 head, linear state over all tokens + %d query rows against all "
                                   "keys; extrapolated to H heads x N rows" % last["rows"]},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


def run_ours(args, wl):
    import numpy as np
    import torch
    import torch.distributed as dist
    from paper_2509_24899_b200 import HybridAttention, binding, workloads as W
    import dataclasses

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; the product path has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # every rank draws its own layer input (independent batches: weak scaling, no exchange step)
    wl_r = rank_workload(wl, rank)
    data = W.generate(wl_r)
    to_dev = lambda b: torch.from_numpy(b.view(np.int16)).cuda().view(torch.bfloat16)
    dev = {k: to_dev(v) for k, v in data.items()}
    weights = {k: v for k, v in dev.items() if k not in ("q", "k", "v")}
    # The step's inputs rotate over several copies in HBM (distinct addresses), so that no step finds its q, k, v
    # in L2 from the step before; three sets of inputs plus the output exceed the 126 MB L2 many times over.
    n_sets = 1 if args.skip_extras else max(1, min(3, int(6e9 // (3 * dev["q"].numel() * 2))))
    sets = [{k: dev[k] for k in ("q", "k", "v")}] + [{k: dev[k].clone() for k in ("q", "k", "v")} for _ in range(n_sets - 1)]
    path = {"tensor": binding.AS_PATH_TENSOR, "simt": binding.AS_PATH_SIMT}[args.path]
    op = HybridAttention.from_workload(wl_r, kernel_path=path)
    out = torch.empty_like(dev["q"])
    stream = torch.cuda.current_stream()
    fw = dict(wq2=weights.get("wq2"), wk2=weights.get("wk2"),
              biases={n: t for n, t in weights.items() if n.startswith("b")} or None)
    counter = [0]

    def step():
        x = sets[counter[0] % n_sets]
        counter[0] += 1
        op.forward(x["q"], x["k"], x["v"], weights["wq"], weights["wk"], out=out, stream=stream, **fw)

    sampler = ClockSampler(local, period_s=0.005)
    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    assert op.last_status() == 0, "device time-out during warm-up"

    binding.as_hybrid_attn_profile_enable(op.handle, True)
    launches0 = binding.as_hybrid_attn_launch_count(op.handle)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler.start()
    barrier()
    sampler.reset()
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    barrier()
    ms = e0.elapsed_time(e1)
    launches = binding.as_hybrid_attn_launch_count(op.handle) - launches0
    kms, kcnt = binding.as_hybrid_attn_profile_read(op.handle)
    binding.as_hybrid_attn_profile_enable(op.handle, False)
    status = op.last_status()
    burst_clocks = sampler.summary()

    # A second, longer region (about two seconds): the same step under the power cap, with the SM clock sampled
    # inside it, so that the line carries a burst and a sustained figure side by side.
    sustained = None
    if not args.skip_extras and args.sustained_s > 0:
        n_sus = max(args.steps, int(args.sustained_s * 1e3 / max(ms / args.steps, 1e-3)))
        sampler.reset()
        barrier()
        e0.record(stream)
        for _ in range(n_sus):
            step()
        e1.record(stream)
        barrier()
        sus_ms = e0.elapsed_time(e1)
        sus_clocks = sampler.summary()
        (sus_ms,) = max_over_ranks([sus_ms], "cuda")
        sustained = {"steps": n_sus, "seconds": sus_ms * 1e-3, "ms_per_step": sus_ms / n_sus,
                     "value": whole_job_value(wl, world, n_sus, sus_ms), "clocks": sus_clocks}
        status = status or op.last_status()

    if args.skip_extras:          # profiling runs: only the device-timed region
        if rank == 0:
            print(json.dumps({"ms_per_step": ms / args.steps, "kernel_ms": kms, "launches": int(launches),
                              "device_status": status, "note": "--skip-extras: no e2e, no cpu baseline"}))
        if world > 1:
            dist.destroy_process_group()
        return 0 if status == 0 else 1

    # end to end: host buffers in, host buffer out, copies inside the timed region
    host = {k: torch.from_numpy(data[k].view(np.int16)).pin_memory() for k in ("q", "k", "v")}
    out_host = torch.empty_like(host["q"]).pin_memory()
    e2e_steps = max(3, min(args.steps, 20))
    for _ in range(2):
        op.forward_host(host["q"], host["k"], host["v"], weights["wq"], weights["wk"], out_host, stream=stream, **fw)
    barrier()
    e0.record(stream)
    for _ in range(e2e_steps):
        op.forward_host(host["q"], host["k"], host["v"], weights["wq"], weights["wk"], out_host, stream=stream, **fw)
    e1.record(stream)
    barrier()
    e2e_ms = e0.elapsed_time(e1)
    sampler.stop()

    ms, e2e_ms = max_over_ranks([ms, e2e_ms], "cuda")
    value = whole_job_value(wl, world, args.steps, ms)
    e2e_value = whole_job_value(wl, world, e2e_steps, e2e_ms)

    rc = 0
    if rank == 0:
        peaks = _peaks()
        n_s = op.n_softmax
        fl = flops_per_layer(wl, n_s)
        q_launches = max(kcnt[binding.AS_KERNEL_QPASS], 1)
        q_ms = kms[binding.AS_KERNEL_QPASS] / q_launches
        k_ms = kms[binding.AS_KERNEL_KPASS] / max(kcnt[binding.AS_KERNEL_KPASS], 1)
        r_ms = kms[binding.AS_KERNEL_REDUCE] / max(kcnt[binding.AS_KERNEL_REDUCE], 1)
        if n_s > 0:
            achieved = fl["qpass"] / (q_ms * 1e-3) / 1e12
            roof = {"bound": "tensor", "kernel": "qpass", "achieved": achieved, "peak": peaks["bf16_tflops"],
                    "unit": "TFLOP/s", "frac": achieved / peaks["bf16_tflops"],
                    "traffic": measured_dram_traffic("qpass_kernel", wl.name),
                    "peak_source": "%s burst bf16 (sustained %s)" % (peaks["source"], peaks["bf16_tflops_sustained"]),
                    "frac_of_nominal_2250": achieved / 2250.0,
                    "frac_of_sustained": (achieved / peaks["bf16_tflops_sustained"]) if peaks.get("bf16_tflops_sustained") else None,
                    "avg_launch_ms": q_ms,
                    "avg_launch_sm_cycles": (q_ms * 1e-3 * burst_clocks["sm_mhz"] * 1e6) if burst_clocks.get("sm_mhz") else None,
                    "flops_per_launch": fl["qpass"]}
        else:       # rate 0: the whole layer is bound by reading q, k, v and writing out
            gbs = bytes_per_layer(wl) / ((k_ms + r_ms + q_ms) * 1e-3) / 1e9
            roof = {"bound": "hbm", "kernel": "kpass+qpass", "achieved": gbs, "peak": peaks["hbm_gbs"],
                    "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"], "traffic": None,
                    "peak_source": peaks["source"]}
        # CPU baseline: the oracle on this machine's host cores, bounded sample
        from oracle import hybrid_attention as O
        cores = os.cpu_count() or 1
        d1 = {k: W.bf16_bits_to_f64(v[:, :1] if k in ("q", "k", "v") else v[:1]) for k, v in data.items()}
        mask = O.softmax_token_mask(wl.grid, wl.block, wl.rate)
        cb = cpu_oracle_rate(wl, d1, mask, budget_s=15.0, heads=1)
        clocks = burst_clocks if burst_clocks.get("samples", 0) >= 2 or sustained is None else sustained["clocks"]
        if sustained is not None:
            sus_tflops = fl["total"] / (sustained["ms_per_step"] * 1e-3) / 1e12
            sustained.update({"tflops": sus_tflops, "frac_of_nominal_2250": sus_tflops / 2250.0,
                              "peak": peaks.get("bf16_tflops_sustained"),
                              "frac_of_sustained_peak": (sus_tflops / peaks["bf16_tflops_sustained"])
                              if peaks.get("bf16_tflops_sustained") else None})
        line = {
            "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": config_of(wl, n_s, world),
            "timing": {"kernel_path": args.path,
                       "l2": "q,k,v,out of a step total %.0f MB > 126 MB L2; inputs rotate over %d sets of buffers"
                             % (bytes_per_layer(wl) / 1e6, n_sets)},
            "tflops": fl["total"] * args.steps / (ms * 1e-3) / 1e12 * 1.0,
            "kernel_ms": {"kpass": k_ms, "reduce": r_ms, "qpass": q_ms},
            "roofline": roof,
            "cpu_baseline": {"value": cb["tokens_per_s"], "unit": "tokens/s", "cores": cores, "kind": "oracle",
                             "sample": "1 head: linear state over all tokens + %d query rows against all keys; "
                                       "extrapolated to %d heads x %d rows" % (cb["rows"], wl.H, wl.N)},
            "e2e": {"value": e2e_value, "unit": "tokens/s",
                    "h2d_bytes_per_step": 3 * wl.B * wl.H * wl.N * wl.d * 2,
                    "d2h_bytes_per_step": wl.B * wl.H * wl.N * wl.d * 2, "steps": e2e_steps},
            "gpu_launches": int(launches),
            "sustained": sustained,
            "clocks": clocks,
            "device_status": status,
        }
        print(json.dumps(line))
        if status != 0:
            rc = 1
    if world > 1:
        dist.destroy_process_group()
    return rc


def run_seq_shard(args, wl):
    """One layer with its TOKENS spread over the ranks (strong scaling): every rank holds a contiguous range of q, k, v
    rows, runs the key stage, takes part in one all-reduce (S, z) and one all-gather (K_S, V_S) over NCCL, and runs the
    query stage on its rows.  Prints one JSON line of its own; the headline line is the unsharded layer."""
    import numpy as np
    import torch
    import torch.distributed as dist
    from paper_2509_24899_b200 import HybridAttention, seq_shard, workloads as W
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; the product path has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    class Alone:                                   # one rank: nothing to exchange
        def all_reduce_sum(self, t):
            return t

        def all_gather_rows(self, t, rows_per_rank):
            return t

    # the layer's softmax tokens from the library's own token rule (a handle for the whole layer)
    whole = HybridAttention.from_workload(wl)
    idx = whole.softmax_indices()
    whole.close()
    op = seq_shard.SeqShardedAttention(wl.B, wl.H, wl.N, wl.d, idx, rank, world, comm=None if world > 1 else Alone(),
                                       phi_dim=wl.F, poly_degree=wl.degree, phi_layers=wl.layers, phi_hidden=wl.hidden_width)
    data = W.generate(wl)                          # the same layer on every rank; each keeps its rows
    to_dev = lambda b: torch.from_numpy(b.view(np.int16)).cuda().view(torch.bfloat16)
    rows = {k: to_dev(np.ascontiguousarray(data[k][:, :, op.n0:op.n1])) for k in ("q", "k", "v")}
    wts = {k: to_dev(v) for k, v in data.items() if k not in ("q", "k", "v")}
    extra = dict(wq2=wts.get("wq2"), wk2=wts.get("wk2"))
    out = torch.empty_like(rows["q"])
    stream = torch.cuda.current_stream()
    step = lambda: op.forward(rows["q"], rows["k"], rows["v"], wts["wq"], wts["wk"], out=out, **extra)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    barrier()
    (ms,) = max_over_ranks([e0.elapsed_time(e1)], "cuda")
    status = op.op.last_status()
    if rank == 0:
        print(json.dumps({"metric": METRIC, "value": wl.B * wl.N * args.steps / (ms * 1e-3), "unit": "tokens/s",
                          "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps,
                          "higher_is_better": True, "scaling": "strong", "dtype": "bf16", "data": "synthetic",
                          "config": dict(config_of(wl, len(idx), world), parallelism="sp%d (token ranges; all-reduce of S, z and "
                                         "all-gather of K_S, V_S per layer)" % world),
                          "exchange_bytes_per_step": {"all_reduce": wl.B * wl.H * wl.F * (wl.d + 1) * 4,
                                                      "all_gather": 2 * wl.B * wl.H * len(idx) * wl.d * 2},
                          "device_status": status}))
    if world > 1:
        dist.destroy_process_group()
    return 0 if status == 0 else 1


def run_stack(args):
    """The 30-layer block-rate stack: one timed layer per distinct rate, per-layer and summed time against
    all layers running full softmax (rate 1).  Prints one JSON line of its own; not the headline line."""
    import numpy as np
    import torch
    from paper_2509_24899_b200 import HybridAttention, workloads as W
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; the product path has no CPU fallback")
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    sched = W.stack_schedule(0)
    per_rate = {}
    stream = torch.cuda.current_stream()
    for rate in W.STACK_RATES:
        wl = W.stack_layer(sched.index(rate))
        data = W.generate(wl)
        dev = {k: torch.from_numpy(v.view(np.int16)).cuda().view(torch.bfloat16) for k, v in data.items()}
        op = HybridAttention.from_workload(wl)
        out = torch.empty_like(dev["q"])
        steps = max(3, args.steps // (10 if rate == 1 else 1))
        for _ in range(3):
            op.forward(dev["q"], dev["k"], dev["v"], dev["wq"], dev["wk"], out=out, stream=stream)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(steps):
            op.forward(dev["q"], dev["k"], dev["v"], dev["wq"], dev["wk"], out=out, stream=stream)
        e1.record(stream)
        torch.cuda.synchronize()
        assert op.last_status() == 0
        per_rate[rate] = {"ms_per_layer": e0.elapsed_time(e1) / steps, "layers": sched.count(rate),
                          "n_softmax": op.n_softmax, "steps": steps}
        del op, dev, out
    total = sum(v["ms_per_layer"] * v["layers"] for v in per_rate.values())
    all_softmax = per_rate[1]["ms_per_layer"] * len(sched)
    # Block-rate selection with the costs just measured and synthetic per-block errors: the same budget
    # as the fixed schedule, spent where the (synthetic) error falls fastest.
    from paper_2509_24899_b200 import binding
    err = W.stack_errors(0)
    cost = [[per_rate[r]["ms_per_layer"] for r in W.STACK_RATES] for _ in sched]
    choice, sel_ms, sel_err = binding.as_select_block_rates(cost, err.tolist(), total)
    fixed_err = float(sum(err[i][W.STACK_RATES.index(r)] for i, r in enumerate(sched)))
    selection = {"budget_ms": total, "selected_ms": sel_ms, "selected_err": sel_err, "fixed_schedule_err": fixed_err,
                 "selected_rates": [W.STACK_RATES[c] for c in choice], "errors": "synthetic"}
    print(json.dumps({"workload": "stack", "schedule": sched, "per_rate": {str(k): v for k, v in per_rate.items()},
                      "stack_ms": total, "all_softmax_ms": all_softmax, "speedup_vs_all_softmax": all_softmax / total,
                      "block_rate_selection": selection, "dtype": "bf16", "data": "synthetic"}))
    return 0


def run_backward(args, wl):
    """The gradient of the value-distillation loss w.r.t. the feature-map weights ("Attention Distillation"): one
    forward that keeps its per-row statistics, then backward_phi, device-timed separately.  One JSON line of its
    own (the headline line is the forward pass); one-layer maps with F = d only."""
    import torch
    from paper_2509_24899_b200 import HybridAttention, workloads as W
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; the product path has no CPU fallback")
    torch.cuda.set_device(0)
    data = W.generate(wl)
    dev = {k: torch.from_numpy(v.view("int16")).cuda().view(torch.bfloat16) for k, v in data.items()}
    y_t = torch.from_numpy(W.teacher_output(wl).view("int16")).cuda().view(torch.bfloat16)
    op = HybridAttention.from_workload(wl)
    out = torch.empty_like(dev["q"])
    aux = torch.empty(wl.B, wl.H, wl.N, 3, dtype=torch.float32, device="cuda")

    def fwd():
        op.forward(dev["q"], dev["k"], dev["v"], dev["wq"], dev["wk"], out=out, aux=aux)

    def bwd():
        return op.backward_phi(dev["q"], dev["k"], dev["v"], dev["wq"], dev["wk"], y_t, out, aux)

    for _ in range(max(args.warmup, 3)):
        fwd(); bwd()
    torch.cuda.synchronize()
    assert op.last_status() == 0, "device time-out during warm-up"
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
    f_ms = b_ms = 0.0
    for _ in range(args.steps):
        ev[0].record(); fwd(); ev[1].record(); bwd(); ev[2].record()
        torch.cuda.synchronize()
        f_ms += ev[0].elapsed_time(ev[1]); b_ms += ev[1].elapsed_time(ev[2])
    dwq, dwk, loss = bwd()
    torch.cuda.synchronize()
    n_l = wl.N - op.n_softmax
    # products of the chain rule per head: dphi_q = g' S^T - (g'.y) z (N x d x F), dW_q (N x F x d), dS (N x F x d),
    # dphi_k = v dS^T + dz (N_L x d x F), dW_k (N_L x F x d); 2 flops per multiply-add
    flops = wl.B * wl.H * 2.0 * wl.F * wl.d * (3 * wl.N + 2 * n_l)
    print(json.dumps({"op": "forward(aux) + backward_phi", "metric": "gradient step of the phi weights", "unit": "ms",
                      "forward_ms": f_ms / args.steps, "backward_ms": b_ms / args.steps, "steps": args.steps,
                      "backward_gflop": flops / 1e9, "backward_tflops": flops / (b_ms / args.steps * 1e-3) / 1e12,
                      "loss": float(loss.item()), "grad_norms": [float(dwq.norm()), float(dwk.norm())],
                      "dtype": ("bf16 operands, fp32 accumulation (tcgen05 kernels)" if wl.d == 128 and wl.F == 128
                                else "bf16 in, fp32 arithmetic (CUDA cores)"), "data": "synthetic",
                      "config": config_of(wl, op.n_softmax, 1), "device_status": op.last_status()}))
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="wan81",
                    help="tiny | wan17 | wan81 | wan161cfg | stack:<layer> | stack (all five rates, summed) | "
                         "wan81_paper_phi | wan81_f256 (the headline layer with wider feature maps)")
    ap.add_argument("--path", default="tensor", choices=["tensor", "simt"],
                    help="kernel path: tcgen05 tensor-core kernels (default) or the fp32 CUDA-core check path")
    ap.add_argument("--sustained-s", type=float, default=2.0,
                    help="length in seconds of the second, power-capped timed region (0 = none)")
    ap.add_argument("--shard", default="batch", choices=["batch", "seq"],
                    help="batch: every rank its own layer input (the headline, weak scaling); seq: one layer with its "
                         "tokens spread over the ranks (strong scaling, two NCCL exchanges per layer)")
    ap.add_argument("--op", default="forward", choices=["forward", "backward"],
                    help="forward: the headline line; backward: forward with statistics + gradient w.r.t. the phi weights")
    ap.add_argument("--skip-extras", action="store_true",
                    help="only the device-timed steps (for profiler runs): no e2e, no CPU baseline")
    args = ap.parse_args()
    from paper_2509_24899_b200 import workloads as W
    if args.workload == "stack":
        return run_stack(args)
    if args.workload.startswith("stack:"):
        wl = W.stack_layer(int(args.workload.split(":")[1]))
    elif args.workload in W.VARIANTS:
        wl = W.VARIANTS[args.workload]
    else:
        wl = W.CONFIGS[args.workload]
    if args.impl == "reference":
        return run_reference(args, wl)
    if args.op == "backward":
        return run_backward(args, wl)
    if args.shard == "seq":
        return run_seq_shard(args, wl)
    return run_ours(args, wl)


if __name__ == "__main__":
    sys.exit(main())

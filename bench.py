#!/usr/bin/env python
"""Benchmark of the sparse drafter linears: microseconds per drafted token at N = 1.

A "step" is one token through every decoder-block linear of the drafter: one call of
``sd2_drafter_step``, a single persistent launch that runs the 4 x ``blocks`` dependent stages
(q|k|v, o, gate|up, down of every block; seven sparse linears per block) separated by grid-wide
barriers, replayed as a CUDA graph.  Default workload: Llama-3.2-1B-shaped drafter, 16
blocks, 50 % unstructured sparsity, one activation row (the configuration the metric is quoted
on).  Every block has its own seeded weights, so one step streams about 1.2 GB of compressed
weights, far more than the 126 MB L2: each launch reads its weights from HBM.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

With ``--gpus N`` > 1 (under torchrun) every rank runs an independent replica of the drafter
(the path does not shard: replicas only); the value is the job's aggregate time per token.
``--impl reference`` times the CPU oracle on the host cores on a bounded sample of the same
workload.  One JSON line is printed by rank 0.
"""

from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2504_08838_b200 import synth  # noqa: E402

METRIC = "sparse drafter linear us/token at N=1"
UNIT = "us/token"
WORKLOADS = {
    "llama-3.2-1b": (2, synth.LLAMA_1B),
    "qwen-2.5-1.5b": (3, synth.QWEN_1P5B),
    "llama-3.2-3b": (4, synth.LLAMA_3B),
}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=50)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama-3.2-1b", choices=sorted(WORKLOADS))
    ap.add_argument("--sparsity", type=float, default=0.5)
    ap.add_argument("--mask", default="bernoulli", choices=["bernoulli", "magnitude", "2:4"],
                    help="mask recipe; 2:4 keeps two of every four columns (sparsity is then 0.5)")
    ap.add_argument("--n", type=int, default=1, help="activation rows per step")
    ap.add_argument("--format", default="auto", choices=["auto", "bitmask", "gap4"])
    ap.add_argument("--blocks", type=int, default=0, help="override the block count (0 = the drafter's)")
    ap.add_argument("--no-dense", action="store_true", help="skip the cuBLAS dense comparison")
    ap.add_argument("--no-cpu", action="store_true", help="skip the timed CPU oracle")
    args = ap.parse_args()
    if args.mask == "2:4":
        args.sparsity = 0.5
    return args


MASK_TEXT = {
    "bernoulli": "%d%% unstructured Bernoulli sparsity",
    "magnitude": "%d%% unstructured sparsity by magnitude, per-row densities spread by Beta(2,2)",
    "2:4": "2:4 sparsity by magnitude (two of every four columns kept)",
}


def config_dict(args, shape, blocks, extra=None):
    cfg = {
        "workload": "%s-shaped drafter, %d blocks x 7 linears (q,k,v,o,gate,up,down), %s, "
                    "bf16 weights N(0,0.02), N=%d activation rows N(0,1)"
                    % (shape.name, blocks,
                       MASK_TEXT[args.mask] % round(100 * args.sparsity) if "%d" in MASK_TEXT[args.mask] else MASK_TEXT[args.mask],
                       args.n),
        "mask": args.mask,
        "blocks": blocks,
        "sparsity": args.sparsity,
        "n_rows": args.n,
        "format": args.format,
        "l2": "no flush needed: each step streams every block's own weights (>1 GB), far more than the 126 MB L2",
    }
    if extra:
        cfg.update(extra)
    return cfg


# ------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------

class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs."""

    REASONS = {
        0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x10: "sync_boost",
        0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown",
        0x100: "display_clock_setting",
    }

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in self.REASONS.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(0.01)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        return {
            "sm_mhz": float(np.median(self.samples)) if self.samples else None,
            "sm_max_mhz": self.max_mhz,
            "reasons": sorted(self.reasons),
            "samples": len(self.samples),
        }


# ------------------------------------------------------------------------------------------
# the CPU oracle as a timed baseline (the only place bench.py executes oracle/)
# ------------------------------------------------------------------------------------------

def time_oracle(shape, cfg_id, density, n_rows, blocks_sample, mask_kind="bernoulli"):
    """Seconds the oracle needs for `blocks_sample` blocks' seven linears (single thread)."""
    from oracle import oracle
    total = 0.0
    for b in range(blocks_sample):
        lin = synth.make_block(cfg_id, b, shape, density, mask_kind)
        for i, (W, m) in enumerate(lin):
            X = synth.make_activations(cfg_id, b, i, n_rows, W.shape[1])
            t0 = time.perf_counter()
            oracle.masked_linear(W, m, X)
            total += time.perf_counter() - t0
    return total


def run_reference(args):
    """The oracle, as it stands, timed on the host cores: exactly --steps timed steps after --warmup
    untimed ones, each a bounded sample of the workload (the leading rows of every linear of one
    block, scaled up to all rows and all blocks), sized so that the whole run takes a few minutes."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg_id, shape = WORKLOADS[args.workload]
    blocks = args.blocks or shape.blocks
    density = 1.0 - args.sparsity
    from oracle import oracle
    oracle.build()
    pool = [synth.make_block(cfg_id, b, shape, density, args.mask) for b in range(min(blocks, 2))]
    xs = [[synth.make_activations(cfg_id, b, i, args.n, W.shape[1]) for i, (W, _) in enumerate(lin)]
          for b, lin in enumerate(pool)]

    def one_block(b, frac):
        total = 0.0
        for i, (W, m) in enumerate(pool[b]):
            rows = max(1, int(round(frac * W.shape[0])))
            t0 = time.perf_counter()
            oracle.masked_linear(W[:rows], m[:rows], xs[b][i])
            total += (time.perf_counter() - t0) * W.shape[0] / rows
        return total

    t_block = one_block(0, 1.0)                               # calibration, not reported
    budget = 150.0 / max(1, args.steps + args.warmup)         # seconds of oracle work per step
    frac = min(1.0, max(budget / t_block, 1.0 / 256))
    for k in range(args.warmup):
        one_block(k % len(pool), frac)
    per_step = [one_block(k % len(pool), frac) * blocks for k in range(args.steps)]
    us = float(np.mean(per_step)) * 1e6 if per_step else float("nan")
    sample_txt = ("per step: the first %.1f %% of the rows of all 7 linears of one block (N=%d), scaled to all rows "
                  "and by %d blocks" % (100 * frac, args.n, blocks))
    line = {
        "impl": "reference", "metric": METRIC, "value": us, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": us / 1e3, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_dict(args, shape, blocks),
        "cpu_baseline": {"value": us, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample_txt},
        "e2e": {"value": us, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------
# the CUDA path
# ------------------------------------------------------------------------------------------

def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        return float(json.load(open(path))["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


def ncu_traffic_ratio():
    """DRAM bytes per algorithmic byte of the dominant kernel, from the committed ncu summary."""
    import re
    name = "stream_kernel_nt1_llama1b_2blocks.md"
    try:
        text = open(os.path.join(ROOT, "profiles", name)).read()
        m = re.search(r"dram_bytes_per_algorithmic_byte = ([0-9.]+)", text)
        return {"dram_bytes_per_algorithmic_byte": float(m.group(1)), "source": "profiles/" + name}
    except Exception:
        return None


def aggregate_replicas(t_step, world, dist, device):
    """Replicas only: every rank runs its own drafter, nothing is exchanged on the data path.
    The step time of the job is the slowest rank's (MAX over ranks); in that time `world` tokens are
    finished, so the time per token of the whole job is max / world.  Returns (max over ranks of
    t_step, 1e3 * that / world): with t_step in ms the second value is microseconds per token."""
    if world > 1:
        import torch
        t = torch.tensor([t_step], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        t_step = float(t.item())
    return t_step, t_step * 1e3 / world


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2504_08838_b200 import binding as sd2

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    sd2.lib()

    cfg_id, shape = WORKLOADS[args.workload]
    blocks = args.blocks or shape.blocks
    density = 1.0 - args.sparsity
    fmt = {"auto": sd2.SD2_FORMAT_AUTO, "bitmask": sd2.SD2_FORMAT_BITMASK, "gap4": sd2.SD2_FORMAT_GAP4}[args.format]
    N = args.n

    # ---- build the drafter: seeded weights -> compressed handles (+ dense copies for cuBLAS)
    t0 = time.time()
    handles, dense = [], []
    comp_bytes = nnz = dense_elems = 0
    for b in range(blocks):
        lin = synth.make_block(cfg_id, b, shape, density, args.mask)
        hs = []
        for i, (W, m) in enumerate(lin):
            hs.append(sd2.sd2_compress(W, m, fmt, sd2.SD2_DTYPE_BF16))
            comp_bytes += hs[-1].compressed_bytes
            nnz += hs[-1].nnz
            dense_elems += W.size
            if not args.no_dense:
                Wm = np.where(m != 0, W, np.uint16(0))
                dense.append(torch.from_numpy(Wm.view(np.int16)).cuda().view(torch.bfloat16))
        handles.append(hs)
    setup_s = time.time() - t0

    x_host = torch.from_numpy(synth.make_activations(cfg_id, 0, 0, N, shape.hidden).view(np.int16).copy()).view(torch.bfloat16).pin_memory()
    x_dev = x_host.cuda()
    ws_bytes = sd2.sd2_block_workspace_bytes(handles[0], N)
    ws = torch.zeros(ws_bytes // 2, dtype=torch.bfloat16, device="cuda")
    acts = [x_dev] + [torch.zeros((N, shape.hidden), dtype=torch.bfloat16, device="cuda") for _ in range(blocks)]
    y_host = torch.zeros((N, shape.hidden), dtype=torch.bfloat16).pin_memory()
    harr = [sd2._handle_array(hs) for hs in handles]
    launches_per_step = (N + 3) // 4          # one persistent launch per panel of at most 4 rows
    drafter = sd2.sd2_drafter_create(handles, n_max=N)
    y_dev = acts[blocks]

    def token():
        sd2.sd2_drafter_step(drafter, acts[0], y_dev)

    def token_blockwise():
        for b in range(blocks):
            sd2.sd2_block_step(handles[b], acts[b], acts[b + 1], ws, handle_array=harr[b])

    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        for _ in range(3):
            token()
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            token()
        # ---- device-resident timing: K graph replays between two events on the launch stream
        for _ in range(max(args.warmup, 3)):
            graph.replay()
        stream.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        sampler = ClockSampler(local)
        sampler.start()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(args.steps):
            graph.replay()
        e1.record(stream)
        stream.synchronize()
        ms_total = e0.elapsed_time(e1)
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        clocks = sampler.stop()

        # ---- end to end: pinned host x -> device, the token, device y -> pinned host, every step
        def e2e_step():
            acts[0].copy_(x_host, non_blocking=True)
            graph.replay()
            y_host.copy_(acts[blocks], non_blocking=True)
            stream.synchronize()
        for _ in range(5):
            e2e_step()
        e2e_steps = min(args.steps, 500)
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            e2e_step()
        e2e_s = (time.perf_counter() - t0) / e2e_steps
        acts[0].copy_(x_host)

        # ---- the same token as one sd2_block_step launch per block (plain stream launches)
        for _ in range(3):
            token_blockwise()
        stream.synchronize()
        e0.record(stream)
        for _ in range(50):
            token_blockwise()
        e1.record(stream)
        stream.synchronize()
        ms_stream = e0.elapsed_time(e1) / 50

        # ---- cuBLAS dense bf16 on the same masked weights, same chaining, same graph treatment
        dense_us = None
        if not args.no_dense:
            hid, kv, inter = shape.hidden, shape.kv, shape.inter
            bufs = {"q": torch.zeros((N, hid), dtype=torch.bfloat16, device="cuda"),
                    "k": torch.zeros((N, kv), dtype=torch.bfloat16, device="cuda"),
                    "v": torch.zeros((N, kv), dtype=torch.bfloat16, device="cuda"),
                    "h": torch.zeros((N, hid), dtype=torch.bfloat16, device="cuda"),
                    "g": torch.zeros((N, inter), dtype=torch.bfloat16, device="cuda"),
                    "u": torch.zeros((N, inter), dtype=torch.bfloat16, device="cuda"),
                    "t": torch.zeros((N, inter), dtype=torch.bfloat16, device="cuda")}
            dacts = [x_dev.clone()] + [torch.zeros((N, hid), dtype=torch.bfloat16, device="cuda") for _ in range(blocks)]

            def dense_token():
                for b in range(blocks):
                    Wq, Wk, Wv, Wo, Wg, Wu, Wd = dense[7 * b:7 * b + 7]
                    torch.matmul(dacts[b], Wq.t(), out=bufs["q"])
                    torch.matmul(dacts[b], Wk.t(), out=bufs["k"])
                    torch.matmul(dacts[b], Wv.t(), out=bufs["v"])
                    torch.matmul(bufs["q"], Wo.t(), out=bufs["h"])
                    torch.matmul(bufs["h"], Wg.t(), out=bufs["g"])
                    torch.matmul(bufs["h"], Wu.t(), out=bufs["u"])
                    torch.mul(torch.nn.functional.silu(bufs["g"]), bufs["u"], out=bufs["t"])
                    torch.matmul(bufs["t"], Wd.t(), out=dacts[b + 1])
            for _ in range(3):
                dense_token()
            stream.synchronize()
            dgraph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(dgraph, stream=stream):
                dense_token()
            for _ in range(10):
                dgraph.replay()
            stream.synchronize()
            dsteps = max(20, args.steps // 4)
            e0.record(stream)
            for _ in range(dsteps):
                dgraph.replay()
            e1.record(stream)
            stream.synchronize()
            dense_us = e0.elapsed_time(e1) / dsteps * 1e3

    ms_step = ms_total / args.steps
    ms_step, us_token = aggregate_replicas(ms_step, world, dist, "cuda")
    e2e_s, e2e_us = aggregate_replicas(e2e_s, world, dist, "cuda")
    e2e_us *= 1e3                                # seconds -> the helper's "x 1e3" gives ms; us needs another 1e3

    if rank == 0:
        peak, peak_src = measured_peak()
        achieved = comp_bytes / (ms_step * 1e-3) / 1e9           # per replica: bytes of one token / its time
        traffic = ncu_traffic_ratio()
        roofline = {
            "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
            "peak_source": peak_src, "frac_of_8TBps_nominal": achieved / 8000.0,
            "kernel": "stream_kernel<%d>" % min(4, 1 << max(0, (min(N, 4) - 1).bit_length())),
            "algorithmic_bytes_per_launch": comp_bytes / launches_per_step,
            "avg_launch_us": ms_step * 1e3 / launches_per_step,
            "traffic": (traffic["dram_bytes_per_algorithmic_byte"] * comp_bytes / launches_per_step) if traffic else None,
            "traffic_source": traffic.get("source") if traffic else None,
        }
        cpu = None
        if not args.no_cpu and N == 1:
            from oracle import oracle
            oracle.build()
            sample = min(blocks, 8)
            sec = time_oracle(shape, cfg_id, density, N, sample, args.mask)
            cpu = {"value": sec * blocks / sample * 1e6, "unit": UNIT, "cores": 1, "kind": "oracle",
                   "sample": "%d of %d blocks (all 7 linears, N=1), one pass, scaled by %d/%d" % (sample, blocks, blocks, sample)}
        line = {
            "metric": METRIC, "value": us_token, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": False, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": config_dict(args, shape, blocks, {
                "parallelism": "replicas x%d" % world, "compressed_bytes_per_token": comp_bytes,
                "bytes_per_kept_weight": comp_bytes / max(nnz, 1), "dense_bf16_bytes_per_token": 2 * dense_elems,
                "timing": "CUDA events around %d CUDA-graph replays of sd2_drafter_step (one persistent launch per token)" % args.steps,
                "setup_seconds": round(setup_s, 1)}),
            "clocks": clocks,
            "e2e": {"value": e2e_us, "unit": UNIT, "h2d_bytes_per_step": int(x_host.numel() * 2),
                    "d2h_bytes_per_step": int(y_host.numel() * 2), "steps": e2e_steps,
                    "how": "wall clock per token: pinned-host x -> device, graph replay, device y -> pinned host, sync"},
            "gpu_launches": launches_per_step * args.steps,
            "roofline": roofline,
            "cpu_baseline": cpu,
            "block_step_launches_us_per_token": ms_stream * 1e3,
            "cublas_dense_bf16_us_per_token": dense_us,
            "speedup_vs_cublas_dense": (dense_us / (ms_step * 1e3)) if dense_us else None,
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

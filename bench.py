#!/usr/bin/env python
"""Benchmark of the decode-attention hot path (append -> split-KV attention -> LSE merge).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME|INDEX]
                    [--impl ours|reference] [--no-others] [--no-graph]

A step is one pass of the whole path over one batch: for every layer of the workload, the
append of the new token's k,v followed by decode attention, through the C ABI.  One JSON
line is printed by rank 0.  With N > 1 (launched by torch.distributed.run) every rank runs
its own batch of the same shape on its own GPU: independent sequences, no data-path
collective, weak scaling; timing is the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2409_04992_b200 import workloads as wl  # noqa: E402

METRIC = "decode_attention_hbm_gbs"
UNIT = "GB/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
L2_BYTES = 126 * 1024 * 1024
DEFAULT_WORKLOAD = 4
BAD_REASONS = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown")


# Small long-context cases of the grouped-head entry point for profiling (about 1 GB of K and V each):
# name: batch, context, block_tokens, kv_heads, q_heads, q_tokens, head_dim
PROFILE_GROUPED = {
    "mha": (4, 16384, 16, 32, 32, 1, 128),
    "gqa8": (16, 16384, 16, 8, 64, 1, 128),
    "gqa4_4new": (16, 16384, 16, 8, 32, 4, 128),
    "d64": (8, 16384, 16, 32, 32, 1, 64),
    "d256": (4, 16384, 16, 16, 16, 1, 256),
}


def parse_args(argv=None):
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default=str(DEFAULT_WORKLOAD))
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--no-others", action="store_true",
                    help="skip the short extra measurements of the other long-context workloads")
    ap.add_argument("--no-graph", action="store_true", help="do not replay the step from a CUDA graph")
    ap.add_argument("--cpu-seconds", type=float, default=15.0,
                    help="CPU budget of the oracle baseline (0 skips it)")
    ap.add_argument("--layers", type=int, default=0,
                    help="override the workload's layer count (profiling a small case)")
    ap.add_argument("--case", default="",
                    help="run one small profiling case instead of the benchmark and print its timing: "
                         "sparse:<workload index>[:<batch>[:<kt block tokens>]] or grouped:<name> "
                         "(names: " + ", ".join(n for n in PROFILE_GROUPED) + ")")
    ap.add_argument("--launches", type=int, default=2, help="calls made by --case")
    ap.add_argument("--sparse-path", type=int, default=0,
                    help="--case sparse: 0 automatic, 1 staged chain, 2 one block per row")
    ap.add_argument("--grouped-path", type=int, default=0,
                    help="grouped entry point: 0 automatic, 1 warp-level MMAs, 2 tcgen05 where the shape allows")
    return ap.parse_args(argv)


def kernel_source_hash() -> str:
    """sha256 of the file that holds the split kernel (identifies the profiled revision)."""
    import hashlib
    path = os.path.join(ROOT, "paper_2409_04992_b200", "csrc", "decode_attention_kernels.cuh")
    with open(path, "rb") as fh:
        return hashlib.sha256(fh.read()).hexdigest()


def profiled_traffic(workload_name: str, algorithmic_bytes: float):
    """DRAM bytes per launch of the split kernel from the committed ncu summary, scaled by
    the algorithmic bytes of this launch; None if the kernel source changed since."""
    try:
        with open(os.path.join(ROOT, "profiles", "split_kernel_traffic.json")) as fh:
            rec = json.load(fh)
        if rec["kernel_source_sha256"] != kernel_source_hash():
            return None
        scale = algorithmic_bytes / rec["algorithmic_bytes_per_launch"]
        return (rec["dram_bytes_read"] + rec["dram_bytes_write"]) * scale
    except Exception:
        return None


def measured_peak_gbs():
    """HBM copy bandwidth measured on this machine, else the documented fallback."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def sub_roofline(algorithmic_bytes: float, seconds: float) -> dict:
    """HBM roofline of one of the extra measurements: algorithmic bytes of a whole step over
    its device time, against the measured copy bandwidth."""
    peak, kind = measured_peak_gbs()
    achieved = algorithmic_bytes / seconds / 1e9
    return {"bound": "hbm", "algorithmic_bytes": algorithmic_bytes, "achieved": achieved, "peak": peak,
            "peak_kind": kind, "unit": UNIT, "frac": achieved / peak}


# ----------------------------------------------------------------------------- ranks

class Ranks:
    """torch.distributed plumbing: barrier and max/sum over ranks (NCCL on GPUs, gloo on CPU)."""

    def __init__(self, n_gpus: int, backend: str | None = None):
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.rank = int(os.environ.get("RANK", "0"))
        self.local_rank = int(os.environ.get("LOCAL_RANK", "0"))
        self.dist = None
        if self.world > 1:
            import torch.distributed as dist
            os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
            if backend is None:
                backend = "nccl" if torch.cuda.is_available() else "gloo"
            kw = {}
            if backend == "nccl":
                torch.cuda.set_device(self.local_rank)
                kw["device_id"] = torch.device("cuda", self.local_rank)
            dist.init_process_group(backend=backend, **kw)
            self.dist = dist
            self.backend = backend
        if n_gpus != self.world and self.rank == 0:
            print(f"[bench] --gpus {n_gpus} but WORLD_SIZE={self.world}: using {self.world}", file=sys.stderr)

    def _tensor(self, x: float):
        dev = "cuda" if (self.dist and self.backend == "nccl") else "cpu"
        return torch.tensor([x], dtype=torch.float64, device=dev)

    def barrier(self):
        if self.dist:
            self.dist.barrier()

    def max(self, x: float) -> float:
        if not self.dist:
            return x
        t = self._tensor(x)
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return float(t.item())

    def sum(self, x: float) -> float:
        if not self.dist:
            return x
        t = self._tensor(x)
        self.dist.all_reduce(t, op=self.dist.ReduceOp.SUM)
        return float(t.item())

    def close(self):
        if self.dist:
            self.dist.destroy_process_group()


def aggregate(ranks: Ranks, units_this_rank: float, seconds_this_rank: float):
    """Whole-job throughput: units of all ranks over the slowest rank's time."""
    seconds = ranks.max(seconds_this_rank)
    units = ranks.sum(units_this_rank)
    return units / seconds, seconds


# ----------------------------------------------------------------------------- clocks

class ClockSampler(threading.Thread):
    """Samples SM clock and clock-event reasons of one GPU while the timed region runs."""

    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake", 0x2: "applications_clocks"}

    def __init__(self, device_index: int, period_s: float = 0.01):
        super().__init__(daemon=True)
        self.period = period_s
        self.samples, self.reasons, self.sm_max, self.power = [], set(), None, []
        self._stop_flag = threading.Event()
        self._h = None
        try:
            import pynvml
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            try:
                self._h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                self._h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self._nv = pynvml
            self.sm_max = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception as exc:  # pragma: no cover - depends on the box
            self.error = repr(exc)

    def run(self):
        if self._h is None:
            return
        nv = self._nv
        getter = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
            nv.nvmlDeviceGetCurrentClocksThrottleReasons
        while not self._stop_flag.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                bits = int(getter(self._h))
                for bit, name in self.REASONS.items():
                    if bits & bit:
                        self.reasons.add(name)
                self.power.append(nv.nvmlDeviceGetPowerUsage(self._h) / 1000.0)
            except Exception:
                pass
            time.sleep(self.period)

    def finish(self) -> dict:
        self._stop_flag.set()
        self.join(timeout=2.0)
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None,
                "sm_max_mhz": self.sm_max, "reasons": sorted(self.reasons),
                "samples": len(self.samples),
                "power_w_max": round(max(self.power), 1) if self.power else None}


# ----------------------------------------------------------------------------- the GPU path

class Layer:
    """Device and pinned-host buffers of one layer's decode step."""

    def __init__(self, case: wl.Case):
        from paper_2409_04992_b200 import binding
        self.case = case
        B, H, D = case.q.shape
        dev = case.q.device
        self.max_len = max(case.max_seq_len, 1)
        self.out = torch.empty((B, H, D), dtype=torch.float16, device=dev)
        self.lse = torch.empty((B, H), dtype=torch.float32, device=dev)
        self.workspace = binding.alloc_workspace(B, H, D, self.max_len, dev)
        # q, k_new, v_new live in one device buffer so that a host caller uploads them in one copy
        self.qkv = torch.stack([case.q, case.k_new, case.v_new]).contiguous()
        case.q, case.k_new, case.v_new = self.qkv[0], self.qkv[1], self.qkv[2]
        self.host_qkv = self.qkv.cpu().pin_memory()
        self.host_out = torch.empty((B, H, D), dtype=torch.float16).pin_memory()
        self.chunk_tokens = binding.plan_chunk_tokens(B, H, self.max_len)
        self.n_splits = binding.plan_num_splits(B, H, self.max_len)
        self.clustered = binding.plan_merges_in_cluster(B, H, self.max_len)
        self.events = None

    @property
    def launches(self) -> int:
        """append + split + merge; no merge kernel with a single chunk, nor for small problems,
        where the chunks of a (sequence, head) merge inside the split kernel as a cluster."""
        return 2 + (1 if self.n_splits > 1 and not self.clustered else 0)

    def run(self, flags):
        from paper_2409_04992_b200 import binding
        c = self.case
        binding.kv_append(c.k_cache, c.v_cache, c.k_new, c.v_new, c.seq_lens, c.block_table, flags)
        if c.block_table is None:
            binding.decode_attention(self.out, self.lse, c.q, c.k_cache, c.v_cache, c.seq_lens,
                                     self.max_len, c.scale, self.workspace, flags)
        else:
            binding.decode_attention_paged(self.out, self.lse, c.q, c.k_cache, c.v_cache,
                                           c.block_table, c.seq_lens, self.max_len, c.scale,
                                           self.workspace, flags)

    def run_from_host(self, flags):
        """The same step as a caller with host-resident q,k,v sees it: the three new vectors
        go up from pinned memory, the attention output comes back (the KV cache stays on the
        device, which is the point of the method: Sec. IV-D)."""
        from paper_2409_04992_b200 import binding
        c = self.case
        binding.decode_step_host(self.host_out, self.host_qkv, self.qkv, self.out, self.lse, c.k_cache,
                                 c.v_cache, c.seq_lens, c.block_table, self.max_len, c.scale,
                                 self.workspace, flags)

    def run_from_host_overlapped(self, flags, compute, upload, download):
        """The same, with the upload and the download on streams of their own, so that a step of
        many layers overlaps layer L+1's upload and layer L-1's download with layer L's kernels."""
        from paper_2409_04992_b200 import binding
        c = self.case
        if self.events is None:                   # torch creates a CUDA event at its first record
            self.events = (torch.cuda.Event(), torch.cuda.Event())
            for e in self.events:
                e.record(compute)
        binding.decode_step_host_overlapped(self.host_out, self.host_qkv, self.qkv, self.out, self.lse,
                                            c.k_cache, c.v_cache, c.seq_lens, c.block_table, self.max_len,
                                            c.scale, self.workspace, flags, compute, upload, download,
                                            self.events[0], self.events[1])

    @property
    def h2d_bytes(self) -> int:
        return self.host_qkv.numel() * self.host_qkv.element_size()

    @property
    def d2h_bytes(self) -> int:
        return self.host_out.numel() * self.host_out.element_size()


def layer_bytes(w: wl.Workload, lens) -> int:
    """Device bytes of one layer's K and V caches."""
    row = w.heads * w.head_dim * 2
    if w.paged:
        blocks = sum(-(-n // w.block_tokens) for n in lens) + w.spare_blocks
        return 2 * blocks * w.block_tokens * row
    return 2 * w.batch * w.s_max * row


def build_layers(w: wl.Workload, device, rank: int):
    """All layers' inputs on the device.  If the caches of every layer do not fit, fewer
    distinct layer pools (each far larger than L2) are cycled through and reported."""
    lens = wl.draw_seq_lens(w)
    per_layer = layer_bytes(w, lens)
    free, _ = torch.cuda.mem_get_info(device)
    distinct = w.layers
    if per_layer * w.layers > 0.85 * free:
        distinct = max(1, min(w.layers, int(0.85 * free // per_layer)))
    layers = [Layer(wl.generate(w, layer=i + 64 * rank, device=str(device), poison=False,
                                seq_lens=lens)) for i in range(distinct)]
    return [layers[i % distinct] for i in range(w.layers)], distinct


_copy_streams = {}


def run_step(layers, flags, from_host=False):
    """One step.  From host buffers, with every layer owning its staging buffers, the copies run
    on two streams of their own (forked from the current stream and joined at the end of the
    step, so the step is still one unit of work on the current stream)."""
    if from_host and len({id(layer) for layer in layers}) == len(layers) and len(layers) > 1:
        compute = torch.cuda.current_stream()
        dev = compute.device
        if dev not in _copy_streams:
            _copy_streams[dev] = (torch.cuda.Stream(dev), torch.cuda.Stream(dev))
        upload, download = _copy_streams[dev]
        if any(layer.events is None for layer in layers):        # creates the events, outside any capture
            for layer in layers:
                if layer.events is None:
                    layer.events = (torch.cuda.Event(), torch.cuda.Event())
                    for e in layer.events:
                        e.record(compute)
        upload.wait_stream(compute)
        download.wait_stream(compute)
        for layer in layers:
            layer.run_from_host_overlapped(flags, compute, upload, download)
        compute.wait_stream(upload)
        compute.wait_stream(download)
        return
    for layer in layers:
        if from_host:
            layer.run_from_host(flags)
        else:
            layer.run(flags)


class L2Flush:
    """Overwrites a buffer larger than L2 so that the next step starts from HBM."""

    def __init__(self, device):
        self.buf = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=device)

    def __call__(self):
        self.buf.fill_(1)


def timed_steps(ranks: Ranks, layers, flags, steps: int, warmup: int, from_host: bool,
                flush, graph: bool, device):
    """W untimed + K timed steps; returns (seconds for the K steps on this rank, clocks)."""
    stream = torch.cuda.current_stream()
    replay = None
    for _ in range(max(warmup, 1) if graph else 0):     # the library's one-time set-up precedes capture
        run_step(layers, flags, from_host)
    if graph:
        g = torch.cuda.CUDAGraph()
        torch.cuda.synchronize()
        with torch.cuda.graph(g):
            run_step(layers, flags, from_host)
        replay = g.replay
    step = replay if replay else (lambda: run_step(layers, flags, from_host))
    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    ranks.barrier()
    sampler = ClockSampler(device.index or 0)
    sampler.start()
    if flush is None:
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record(stream)
        for _ in range(steps):
            step()
        t1.record(stream)
        torch.cuda.synchronize()
        seconds = t0.elapsed_time(t1) / 1e3
    else:
        pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
                 for _ in range(steps)]
        for a, b in pairs:
            flush()
            a.record(stream)
            step()
            b.record(stream)
        torch.cuda.synchronize()
        seconds = sum(a.elapsed_time(b) for a, b in pairs) / 1e3
    clocks = sampler.finish()
    ranks.barrier()
    return seconds, clocks


def split_kernel_seconds(layers, flags, steps: int, flush):
    """Average duration of one split-KV kernel launch, from events the library records
    around that launch on the stream it runs on (same workload and launch shape as the
    timed region)."""
    from paper_2409_04992_b200 import binding
    before, after = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    stream = torch.cuda.current_stream()
    before.record(stream)
    after.record(stream)
    torch.cuda.synchronize()
    total, count = 0.0, 0
    binding.set_timing_events(before, after)
    try:
        for _ in range(steps):
            for layer in layers:
                if flush is not None:
                    flush()
                layer.run(flags)
                torch.cuda.synchronize()
                total += before.elapsed_time(after) / 1e3
                count += 1
    finally:
        binding.set_timing_events(None, None)
    return total / max(count, 1)


# ----------------------------------------------------------------------------- the CPU oracle

def oracle_sample(w: wl.Workload, target_seconds: float):
    """A bounded sample of the workload for the CPU oracle: full-length sequences of the
    workload's own length distribution and layout, but fewer sequences and heads, sized
    from a short calibration so that one pass takes about `target_seconds`."""
    import numpy as np
    from oracle import capi

    threads = capi.num_threads()
    probe = w.replace(batch=1, heads=threads, len_lo=2048, len_hi=2048,
                      s_max=2048 if not w.paged else 0)
    c = wl.generate(probe, poison=False)
    table = None if c.block_table is None else c.block_table.numpy()
    args = (c.q.numpy(), c.k_cache.numpy(), c.v_cache.numpy(), np.array(c.seq_lens_host), c.scale)
    capi.decode_attention(*args, block_table=table)
    t0 = time.perf_counter()
    capi.decode_attention(*args, block_table=table)
    rate = threads * 2048 / (time.perf_counter() - t0)           # (token, head) rows per second

    mean_len = (w.len_lo + w.len_hi) / 2
    pairs = max(1, int(target_seconds * rate / mean_len))
    if pairs < threads:
        batch, heads = 1, min(w.heads, pairs)
    else:
        batch = max(1, min(w.batch, pairs // threads))
        heads = min(w.heads, max(threads, pairs // batch))
    sample = w.replace(batch=batch, heads=heads, layers=1)
    lens = wl.draw_seq_lens(w)[:batch]
    case = wl.generate(sample, poison=False, seq_lens=lens)
    return case, threads


def oracle_pass(case: wl.Case):
    """One append + attention pass of the oracle; returns seconds."""
    import numpy as np
    from oracle import capi

    table = None if case.block_table is None else case.block_table.numpy()
    lens = np.array(case.seq_lens_host, dtype=np.int32)
    k, v = case.k_cache.numpy(), case.v_cache.numpy()
    t0 = time.perf_counter()
    capi.kv_append(k, v, case.k_new.numpy(), case.v_new.numpy(), lens, block_table=table)
    out, _, _ = capi.decode_attention(case.q.numpy(), k, v, lens, case.scale, block_table=table)
    case.oracle_out = out                         # kept for the parity figure of cpu_baseline
    return time.perf_counter() - t0


def sample_text(case: wl.Case) -> str:
    w = case.workload
    return (f"{w.batch} of {wl.by_name(str(w.index)).batch} sequences x {w.heads} of "
            f"{wl.HEADS_13B} heads x 1 layer, full lengths {case.seq_lens_host}, "
            f"{w.layout} layout, append + attention")


def device_output_of_sample(case: wl.Case, device) -> torch.Tensor:
    """The CUDA path's output on the oracle's sample (its own copy of the same bits)."""
    from paper_2409_04992_b200 import binding
    moved = {k: (v.to(device) if isinstance(v, torch.Tensor) else v) for k, v in case.__dict__.items()
             if k != "oracle_out"}
    dev = wl.Case(**moved)
    B, H, D = dev.q.shape
    out = torch.empty((B, H, D), dtype=torch.float16, device=device)
    ws = binding.alloc_workspace(B, H, D, dev.max_seq_len, device)
    binding.kv_append(dev.k_cache, dev.v_cache, dev.k_new, dev.v_new, dev.seq_lens, dev.block_table)
    if dev.block_table is None:
        binding.decode_attention(out, None, dev.q, dev.k_cache, dev.v_cache, dev.seq_lens,
                                 dev.max_seq_len, dev.scale, ws)
    else:
        binding.decode_attention_paged(out, None, dev.q, dev.k_cache, dev.v_cache, dev.block_table,
                                       dev.seq_lens, dev.max_seq_len, dev.scale, ws)
    torch.cuda.synchronize()
    return out.cpu()


def cpu_baseline(w: wl.Workload, seconds: float, device=None) -> dict:
    case, threads = oracle_sample(w, seconds)
    got = device_output_of_sample(case, device) if device is not None else None
    first = oracle_pass(case)
    passes = 1 + max(0, min(30, int(seconds / max(first, 1e-3)) - 1))   # fill the budget, bounded
    elapsed = first + sum(oracle_pass(case) for _ in range(passes - 1))
    used = min(threads, case.workload.batch * case.workload.heads)
    return {"value": case.kv_bytes_read * passes / elapsed / 1e9, "unit": UNIT, "cores": used,
            "kind": "oracle", "sample": f"{passes} passes over " + sample_text(case),
            "seconds": round(elapsed, 2),
            "kv_tokens_per_s": case.kv_tokens * passes * case.workload.heads / wl.HEADS_13B / elapsed,
            **({} if got is None else {"gpu_vs_oracle_on_sample": parity_figures(got, case.oracle_out)})}


def parity_figures(got_fp16: torch.Tensor, want) -> dict:
    """Largest absolute error, and largest relative error over exact values that are normal fp16."""
    import numpy as np
    g = got_fp16.numpy().astype(np.float64)
    diff = np.abs(g - want)
    big = np.abs(want) >= 2.0 ** -14
    return {"max_abs": float(diff.max()), "max_rel": float((diff[big] / np.abs(want[big])).max()),
            "bounds": {"max_abs": 2e-3, "max_rel": 1e-2}, "elements": int(diff.size)}


def reference_arm(args, world: int) -> None:
    """--impl reference: the CPU oracle, as it stands, timed on host cores (rank 0 only)."""
    w = wl.by_name(args.workload)
    per_step = min(3.0, 120.0 / max(args.steps + args.warmup, 1))
    case, threads = oracle_sample(w, per_step)
    for _ in range(args.warmup):
        oracle_pass(case)
    seconds = sum(oracle_pass(case) for _ in range(args.steps))
    used = min(threads, case.workload.batch * case.workload.heads)
    value = case.kv_bytes_read * args.steps / seconds / 1e9
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": seconds / args.steps * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "sample": sample_text(case)},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": used, "kind": "oracle",
                             "sample": sample_text(case)},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------- main

def measure_workload(w: wl.Workload, ranks: Ranks, device, steps: int, warmup: int,
                     graph: bool, with_e2e: bool):
    """Device-resident timing (+ the split kernel alone, + the host-buffer variant)."""
    layers, distinct = build_layers(w, device, ranks.rank)
    flags = torch.zeros(1, dtype=torch.int32, device=device)
    step_bytes = sum(layer.case.kv_bytes_read for layer in layers)
    step_tokens = sum(layer.case.kv_tokens for layer in layers)
    fits_l2 = layer_bytes(w, layers[0].case.seq_lens_host) * distinct <= 2 * L2_BYTES
    flush = L2Flush(device) if fits_l2 else None

    seconds, clocks = timed_steps(ranks, layers, flags, steps, warmup, False, flush, graph, device)
    if any(r in clocks["reasons"] for r in BAD_REASONS):           # rejected: measure once more
        seconds, clocks = timed_steps(ranks, layers, flags, steps, warmup, False, flush, graph, device)
        clocks["remeasured"] = True
    gbs, job_seconds = aggregate(ranks, step_bytes * steps / 1e9, seconds)
    tokens_per_s = ranks.sum(step_tokens * steps) / job_seconds

    split_s = split_kernel_seconds(layers, flags, max(1, min(steps, 5)), flush)
    split_bytes = step_bytes / len(layers)            # one launch reads one layer's K and V once
    res = {"gbs": gbs, "kv_tokens_per_s": tokens_per_s, "ms_per_step": job_seconds / steps * 1e3,
           "clocks": clocks, "distinct_layer_pools": distinct, "flush": flush is not None,
           "split_seconds": split_s, "split_bytes": split_bytes,
           "launches_per_step": sum(layer.launches for layer in layers),
           "chunk_tokens": layers[0].chunk_tokens, "n_splits": layers[0].n_splits,
           "kv_bytes_per_step": step_bytes, "flags": int(flags.item())}
    if with_e2e:
        e2e_s, _ = timed_steps(ranks, layers, flags, steps, warmup, True, flush, graph, device)
        e2e_gbs, _ = aggregate(ranks, step_bytes * steps / 1e9, e2e_s)
        res["e2e"] = {"value": e2e_gbs, "unit": UNIT,
                      "h2d_bytes_per_step": sum(layer.h2d_bytes for layer in layers),
                      "d2h_bytes_per_step": sum(layer.d2h_bytes for layer in layers)}
    del layers
    torch.cuda.empty_cache()
    return res


def measure_sparse(w: wl.Workload, device, steps: int, r: int = 16, keep: float = 0.125,
                   window: int = 16, kt_block_tokens: int = 256) -> dict:
    """One layer of `w` through the sparse (Algorithm 1) entry points next to the dense ones on
    the same data: append + attention per step, CUDA events, inputs far larger than L2."""
    from paper_2409_04992_b200 import binding
    case = wl.generate(w.replace(layers=1), device=str(device), poison=False)
    state = wl.make_sparf_state(case, keep, kt_block_tokens)
    B, H, D = case.q.shape
    max_len, max_k = case.max_seq_len, max(state.k_tokens_host)
    out = torch.empty((B, H, D), dtype=torch.float16, device=device)
    lse = torch.empty((B, H), dtype=torch.float32, device=device)
    flags = torch.zeros(1, dtype=torch.int32, device=device)
    ws_dense = binding.alloc_workspace(B, H, D, max_len, device)
    ws_sparse = torch.empty(binding.sparf_workspace_bytes(B, H, D, max_len, max_k), dtype=torch.uint8,
                            device=device)

    def dense():
        binding.kv_append(case.k_cache, case.v_cache, case.k_new, case.v_new, case.seq_lens,
                          case.block_table, flags)
        binding.decode_attention_paged(out, lse, case.q, case.k_cache, case.v_cache, case.block_table,
                                       case.seq_lens, max_len, case.scale, ws_dense, flags)

    def sparse():
        binding.sparf_append(case.k_cache, case.v_cache, state.kt_pool, state.v_sum, case.k_new,
                             case.v_new, case.seq_lens, case.block_table, state.kt_block_table, flags)
        binding.sparf_decode_attention(out, None, None, case.q, case.k_cache, case.v_cache,
                                       state.kt_pool, state.v_sum, case.block_table,
                                       state.kt_block_table, case.seq_lens, state.k_tokens, max_len,
                                       max_k, r, window, case.scale, ws_sparse, flags)

    def timed(fn):
        for _ in range(3):
            fn()
        a, z = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(steps):
            fn()
        z.record()
        torch.cuda.synchronize()
        return a.elapsed_time(z) / 1e3 / steps

    t_dense, t_sparse = timed(dense), timed(sparse)
    moved = case.kv_tokens * H * r * 2 + sum(state.k_tokens_host) * H * 2 * D * 2
    return {"r": r, "keep_fraction": keep, "local_window": window,
            "kt_block_tokens": kt_block_tokens, "ms_per_step": t_sparse * 1e3,
            "dense_ms_per_step": t_dense * 1e3, "speedup_over_dense": t_dense / t_sparse,
            "kv_tokens_per_s": case.kv_tokens / t_sparse,
            "algorithmic_bytes": moved, "algorithmic_gbs": moved / t_sparse / 1e9,
            "roofline": sub_roofline(moved, t_sparse),
            "status_flags": int(flags.item())}


def measure_bulk_append(device, steps: int = 10, batch: int = 16, new_tokens: int = 4096) -> dict:
    """Prefill-style append of `new_tokens` tokens per sequence into a paged cache (T=32):
    bytes read plus bytes written per second, comparable with a device-to-device copy."""
    from paper_2409_04992_b200 import binding
    w = wl.STANDARD[4].replace(batch=batch, len_lo=new_tokens, len_hi=new_tokens, layers=1)
    case = wl.generate(w, device=str(device), poison=False)
    gen = torch.Generator(device=device)
    gen.manual_seed(wl.BASE_SEED + 77)
    fresh = [torch.randn((batch, new_tokens, w.heads, w.head_dim), dtype=torch.float32, device=device,
                         generator=gen).to(torch.float16) for _ in range(2)]
    new_lens = torch.full((batch,), new_tokens, dtype=torch.int32, device=device)
    flags = torch.zeros(1, dtype=torch.int32, device=device)

    def step():
        binding.kv_append_bulk(case.k_cache, case.v_cache, fresh[0], fresh[1], case.seq_lens, new_lens,
                               case.block_table, flags)

    for _ in range(3):
        step()
    a, z = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    a.record()
    for _ in range(steps):
        step()
    z.record()
    torch.cuda.synchronize()
    seconds = a.elapsed_time(z) / 1e3 / steps
    moved = 2 * 2 * fresh[0].numel() * 2                      # K and V, read and written, fp16
    return {"tokens_per_sequence": new_tokens, "batch": batch, "ms_per_step": seconds * 1e3,
            "read_plus_write_gbs": moved / seconds / 1e9, "roofline": sub_roofline(moved, seconds),
            "status_flags": int(flags.item())}


GROUPED_SHAPES = [
    # name, batch, context, block_tokens, kv_heads, q_heads, q_tokens, head_dim
    ("gqa8_ctx16k_b64_paged16", 64, 16384, 16, 8, 64, 1, 128),
    ("gqa4_ctx128k_b8_paged64", 8, 131072, 64, 8, 32, 1, 128),
    ("mha_4new_tokens_ctx16k_b16_paged16", 16, 16384, 16, 40, 40, 4, 128),
    ("mha_d64_ctx16k_b32_paged16", 32, 16384, 16, 32, 32, 1, 64),
    ("mha_d256_ctx16k_b16_paged16", 16, 16384, 16, 16, 16, 1, 256),
]


def measure_grouped(device, steps: int = 20) -> dict:
    """The grouped-head / multi-token / other-head-size entry point on a few long-context
    shapes: fp16 K+V bytes read per second (each input several GB, far beyond L2).  Two passes
    over the shapes: `steps` back-to-back steps each, then about 0.4 s of them each (the figure
    a serving loop sees, at the clock the power cap settles on); the short runs all come first,
    so that none of them starts on a GPU the previous shape's long run has just heated."""
    from paper_2409_04992_b200 import binding
    results = {}
    for sustained in (False, True):
        for name, batch, ctx, tokens, kv_heads, q_heads, q_tokens, dim in GROUPED_SHAPES:
            w = wl.Workload(name, 7, batch=batch, len_lo=ctx, len_hi=ctx, layout="paged",
                            block_tokens=tokens, heads=kv_heads, head_dim=dim)
            g = wl.generate_grouped(w, q_tokens, q_heads, device=str(device))
            c = g.base
            flags = torch.zeros(1, dtype=torch.int32, device=device)
            out = torch.empty_like(g.q)
            ws = torch.empty(binding.grouped_workspace_bytes(batch, q_tokens, q_heads, kv_heads, dim, ctx),
                             dtype=torch.uint8, device=device)

            def step():
                binding.kv_append_bulk(c.k_cache, c.v_cache, g.k_new, g.v_new, c.seq_lens, g.new_lens,
                                       c.block_table, flags)
                binding.decode_attention_grouped(out, None, g.q, c.k_cache, c.v_cache, c.block_table,
                                                 c.seq_lens, ctx, c.scale, ws, flags)

            for _ in range(5):
                step()
            a, z = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            kv_bytes = batch * ctx * kv_heads * dim * 2 * 2
            count = max(steps, int(0.4 / (results[name]["ms_per_step"] / 1e3))) if sustained else steps
            torch.cuda.synchronize()
            a.record()
            for _ in range(count):
                step()
            z.record()
            torch.cuda.synchronize()
            seconds = a.elapsed_time(z) / 1e3 / count
            if sustained:
                results[name]["sustained"] = {"value": kv_bytes / seconds / 1e9, "unit": UNIT, "steps": count}
                results[name]["status_flags"] |= int(flags.item())
            else:
                results[name] = {"value": kv_bytes / seconds / 1e9, "unit": UNIT, "ms_per_step": seconds * 1e3,
                                 "steps": count, "kv_bytes_per_step": kv_bytes,
                                 "query_rows_per_kv_head": q_heads // kv_heads * q_tokens,
                                 "roofline": sub_roofline(kv_bytes, seconds),
                                 "kernel": {1: "grouped_attn_split_kernel (warp-level mma.sync)",
                                            2: "grouped_attn_umma_kernel (tcgen05, tensor memory, tensor-map copies)"}.get(
                                                binding.grouped_path_for(dim, tokens), "?"),
                                 "status_flags": int(flags.item())}
            del g, c, out, ws
            torch.cuda.empty_cache()
    return results


def head_sharded_result(ranks: Ranks, units_this_rank: float, seconds_this_rank: float, heads_this_rank: int,
                        total_heads: int, max_abs_error) -> dict:
    """Whole-instance figures of the head-sharded section from per-rank measurements: bytes of
    all ranks over the slowest rank's time (one model instance, strong scaling)."""
    gbs, seconds = aggregate(ranks, units_this_rank, seconds_this_rank)
    heads = ranks.sum(float(heads_this_rank))
    return {"value": gbs, "unit": UNIT, "seconds": seconds, "scaling": "strong",
            "heads_covered": int(round(heads)), "total_heads": total_heads,
            "max_abs_vs_single_gpu": max_abs_error}


def measure_head_sharded(ranks: Ranks, device, steps: int = 20) -> dict:
    """One model instance spread over the ranks the way the paper spreads it over drives
    (Sec. IV-D): one layer of the default workload, batch 16, the 40 heads split over the ranks,
    every rank's KV cache holding only its heads, outputs exchanged by the fused all-gather
    (peer stores of the last kernel into every rank's buffer in symmetric memory).  Only run
    with more than one rank; any failure is returned as text instead of raised, so that it
    cannot take the weak-scaling number down with it."""
    try:
        from paper_2409_04992_b200 import binding, sharding
        w = wl.STANDARD[4].replace(layers=1)
        case = wl.generate(w, device=str(device), poison=False)            # the same bits on every rank
        B, H, D = case.q.shape
        off, cnt = sharding.head_shard(H, ranks.world, ranks.rank)
        q, k_new, v_new = (sharding.take_heads(t, off, cnt) for t in (case.q, case.k_new, case.v_new))
        k_cache = sharding.take_heads(case.k_cache, off, cnt)
        v_cache = sharding.take_heads(case.v_cache, off, cnt)
        peers = sharding.PeerOutputs(B, H, D)
        flags = torch.zeros(1, dtype=torch.int32, device=device)
        max_len = case.max_seq_len
        ws = torch.empty(binding.allgather_workspace_bytes(B, cnt, D, max_len), dtype=torch.uint8, device=device)

        def step():
            binding.kv_append(k_cache, v_cache, k_new, v_new, case.seq_lens, case.block_table, flags)
            binding.decode_attention_allgather(peers.addresses, None, q, k_cache, v_cache, case.block_table,
                                               case.seq_lens, off, H, max_len, case.scale, ws, flags)
            peers.barrier()                        # every rank's rows have landed everywhere

        for _ in range(5):
            step()
        torch.cuda.synchronize()
        ranks.barrier()
        a, z = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(steps):
            step()
        z.record()
        torch.cuda.synchronize()
        ranks.barrier()
        seconds = a.elapsed_time(z) / 1e3
        # rank 0 also runs all heads alone and compares its gathered buffer with that
        error = None
        if ranks.rank == 0:
            out = torch.empty((B, H, D), dtype=torch.float16, device=device)
            full_ws = binding.alloc_workspace(B, H, D, max_len, device)
            binding.kv_append(case.k_cache, case.v_cache, case.k_new, case.v_new, case.seq_lens, case.block_table, flags)
            binding.decode_attention_paged(out, None, case.q, case.k_cache, case.v_cache, case.block_table,
                                           case.seq_lens, max_len, case.scale, full_ws, flags)
            torch.cuda.synchronize()
            error = float((out.float() - peers.local.float()).abs().max())
        shard_bytes = case.kv_bytes_read * cnt / H
        res = head_sharded_result(ranks, shard_bytes * steps / 1e9, seconds, cnt, H, error)
        res["ms_per_step"] = res.pop("seconds") / steps * 1e3
        res["status_flags"] = int(flags.item())
        return res
    except Exception as exc:                       # noqa: BLE001 - reported, never fatal
        return {"error": f"{type(exc).__name__}: {exc}"[:400]}


def run_case(spec: str, launches: int, device, sparse_path: int = 0, grouped_path: int = 0) -> dict:
    """One small case of the sparse or the grouped entry point, `launches` calls back to back
    (what the ncu commands under profiles/ run)."""
    from paper_2409_04992_b200 import binding
    kind, _, rest = spec.partition(":")
    binding.set_sparse_path(sparse_path)
    binding.set_grouped_path(grouped_path)
    flags = torch.zeros(1, dtype=torch.int32, device=device)
    a, z = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if kind == "sparse":
        parts = rest.split(":")
        w = wl.STANDARD[int(parts[0])].replace(layers=1)
        if len(parts) > 1 and parts[1]:
            w = w.replace(batch=int(parts[1]))
        kt_tokens = int(parts[2]) if len(parts) > 2 else 256
        case = wl.generate(w, device=str(device), poison=False)
        state = wl.make_sparf_state(case, 0.125, kt_tokens)
        B, H, D = case.q.shape
        max_len, max_k = case.max_seq_len, max(state.k_tokens_host)
        out = torch.empty((B, H, D), dtype=torch.float16, device=device)
        ws = torch.empty(binding.sparf_workspace_bytes(B, H, D, max_len, max_k), dtype=torch.uint8, device=device)

        def call():
            binding.sparf_decode_attention(out, None, None, case.q, case.k_cache, case.v_cache, state.kt_pool,
                                           state.v_sum, case.block_table, state.kt_block_table, case.seq_lens,
                                           state.k_tokens, max_len, max_k, 16, 16, case.scale, ws, flags)
        moved = case.kv_tokens * H * 16 * 2 + sum(state.k_tokens_host) * H * 2 * D * 2
        name = f"sparse {w.name} batch {w.batch} kt block {kt_tokens}"
    elif kind == "grouped":
        batch, ctx, tokens, kv_heads, q_heads, q_tokens, dim = PROFILE_GROUPED[rest]
        w = wl.Workload(rest, 7, batch=batch, len_lo=ctx, len_hi=ctx, layout="paged", block_tokens=tokens,
                        heads=kv_heads, head_dim=dim)
        g = wl.generate_grouped(w, q_tokens, q_heads, device=str(device))
        c = g.base
        out = torch.empty_like(g.q)
        ws = torch.empty(binding.grouped_workspace_bytes(batch, q_tokens, q_heads, kv_heads, dim, ctx),
                         dtype=torch.uint8, device=device)
        binding.kv_append_bulk(c.k_cache, c.v_cache, g.k_new, g.v_new, c.seq_lens, g.new_lens, c.block_table, flags)

        def call():
            binding.decode_attention_grouped(out, None, g.q, c.k_cache, c.v_cache, c.block_table, c.seq_lens,
                                             ctx, c.scale, ws, flags)
        moved = batch * ctx * kv_heads * dim * 4
        name = f"grouped {rest}"
    else:
        raise ValueError(f"unknown --case {spec!r}")
    torch.cuda.synchronize()
    a.record()
    for _ in range(launches):
        call()
    z.record()
    torch.cuda.synchronize()
    ms = a.elapsed_time(z) / launches
    return {"case": name, "launches": launches, "ms_per_call_first_calls_included": ms,
            "algorithmic_bytes": moved, "algorithmic_gbs": moved / ms / 1e6, "status_flags": int(flags.item())}


def main(argv=None) -> int:
    args = parse_args(argv)
    if args.impl == "reference":          # CPU only: no process group; ranks other than 0 do nothing
        if int(os.environ.get("RANK", "0")) == 0:
            reference_arm(args, int(os.environ.get("WORLD_SIZE", "1")))
        return 0
    ranks = Ranks(args.gpus)
    try:
        from paper_2409_04992_b200 import binding, build
        if not build.is_current() and ranks.local_rank == 0:
            build.build()
        ranks.barrier()
        binding.load()
        if not torch.cuda.is_available():
            raise RuntimeError("bench.py needs a CUDA device: the path has no CPU fallback")
        device = torch.device("cuda", ranks.local_rank)
        torch.cuda.set_device(device)
        if args.case:
            if ranks.rank == 0:
                print(json.dumps(run_case(args.case, args.launches, device, args.sparse_path, args.grouped_path)), flush=True)
            return 0
        w = wl.by_name(args.workload)
        if args.layers > 0:
            w = w.replace(layers=args.layers)
        graph = not args.no_graph
        main_res = measure_workload(w, ranks, device, args.steps, args.warmup, graph, True)

        peak, peak_kind = measured_peak_gbs()
        achieved = main_res["split_bytes"] / main_res["split_seconds"] / 1e9
        line = {
            "metric": METRIC, "value": main_res["gbs"], "unit": UNIT, "n_gpus": ranks.world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": main_res["ms_per_step"],
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic", "impl": "ours",
            "config": {"workload": w.name, "batch_per_gpu": w.batch, "heads": w.heads,
                       "head_dim": w.head_dim, "layers": w.layers, "layout": w.layout,
                       "block_tokens": w.block_tokens, "seq_lens": f"uniform[{w.len_lo},{w.len_hi}]",
                       "kv_dtype": "fp16", "kv_bytes_per_step": main_res["kv_bytes_per_step"],
                       "distinct_layer_pools": main_res["distinct_layer_pools"],
                       "chunk_tokens": main_res["chunk_tokens"], "n_splits": main_res["n_splits"],
                       "cuda_graph": graph,
                       "l2": "flushed between steps" if main_res["flush"] else
                             "inputs larger than L2 (each layer's KV is read once per step)"},
            "kv_tokens_per_s": main_res["kv_tokens_per_s"],
            "pct_of_nominal_8TBs": 100.0 * main_res["gbs"] / ranks.world / NOMINAL_HBM_GBS,
            "pct_of_measured_copy": 100.0 * main_res["gbs"] / ranks.world / peak,
            "clocks": main_res["clocks"], "e2e": main_res["e2e"],
            "gpu_launches": main_res["launches_per_step"] * args.steps,
            "status_flags": main_res["flags"],
            "roofline": {"kernel": "decode_attn_split_kernel", "bound": "hbm",
                         "achieved": achieved, "peak": peak, "peak_kind": peak_kind,
                         "unit": UNIT, "frac": achieved / peak,
                         "peak_note": "the peak is a copy (read + write); a read-only stream such as this "
                                      "kernel can exceed it, so frac > 1 is possible and is not a ceiling",
                         "traffic": profiled_traffic(w.name, main_res["split_bytes"]),
                         "algorithmic_bytes_per_launch": main_res["split_bytes"],
                         "avg_launch_ms": main_res["split_seconds"] * 1e3},
        }
        if ranks.world > 1:
            line["head_sharded"] = measure_head_sharded(ranks, device)
        if ranks.rank == 0 and ranks.world == 1 and args.cpu_seconds > 0:
            line["cpu_baseline"] = cpu_baseline(w, args.cpu_seconds, device)
        if not args.no_others and ranks.world == 1:
            others = {}
            for idx in (0, 1, 2, 3):
                if idx == w.index:
                    continue
                o = wl.STANDARD[idx]
                r = measure_workload(o, ranks, device, 20, 3, False, False)
                others[o.name] = {
                    "value": r["gbs"], "unit": UNIT, "ms_per_step": r["ms_per_step"],
                    "kv_tokens_per_s": r["kv_tokens_per_s"],
                    "pct_of_nominal_8TBs": 100.0 * r["gbs"] / NOMINAL_HBM_GBS,
                    "pct_of_measured_copy": 100.0 * r["gbs"] / peak,
                    "split_kernel_gbs": r["split_bytes"] / r["split_seconds"] / 1e9,
                    "chunk_tokens": r["chunk_tokens"], "l2_flushed_between_steps": r["flush"],
                    "sm_mhz": r["clocks"]["sm_mhz"],
                    "reasons": r["clocks"]["reasons"]}
            line["other_workloads"] = others
            line["bulk_append"] = measure_bulk_append(device)
            line["grouped_attention"] = measure_grouped(device)
            line["sparse_attention"] = {wl.STANDARD[i].name: measure_sparse(wl.STANDARD[i], device, 10)
                                        for i in (2, 3, 4)}      # index 4: one of its layers
        if ranks.rank == 0:
            print(json.dumps(line), flush=True)
        return 0
    finally:
        ranks.close()


if __name__ == "__main__":
    sys.exit(main())

"""Benchmark of the Stream hot path (mask build + block-sparse attention) on synthetic inputs.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

One step = one pass of the whole path over one layer-shaped batch: stream_build_mask followed by
stream_sparse_attention. The headline workload is the 128k-token chain-of-thought-shaped layer
(32 query / 8 kv heads, d = 128, bf16, block 64, k = 32). Prints ONE JSON line (rank 0).

N > 1 (under torchrun): every rank processes its own independent layer (different seed); there is
no data-path collective, so scaling is weak and the value is the sum over ranks divided by the
slowest rank's time.

``--impl reference`` times the CPU oracle (the plain definition the library is tested against) on
the host cores, on a bounded sample of rows per step.
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

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "stream_query_token_heads_per_s"
UNIT = "query-token-heads/s"
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1400.0  # sustained figure of an earlier measurement on this kind of GPU


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cot_layer_128k")
    ap.add_argument("--T", type=int, default=0, help="override the workload's context length")
    ap.add_argument("--kernels", default="auto", choices=["auto", "generic", "tensor"], help="library kernel choice")
    ap.add_argument("--k-sparsity", type=float, default=0.0,
                    help="build the mask with k per query block from this effective sparsity (0 = one k)")
    ap.add_argument("--k-list", default="", help="comma-separated k values: time the several-k mask build (one JSON line, masks only)")
    ap.add_argument("--block-q", type=int, default=0,
                    help="1: time the per-token mask build (block_q = 1, masks only) instead of the step")
    ap.add_argument("--extras", action="store_true",
                    help="instead of the benchmark line: time the analysis kernels (vertical scores, mask subtraction) and "
                         "the several-k build on the workload's masks, each against the HBM peak (one JSON object)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sweep", action="store_true", help="leave the short scaling sweep out of the line")
    ap.add_argument("--cpu-seconds", type=float, default=15.0, help="target CPU time of the oracle sample")
    ap.add_argument("--sweep", action="store_true",
                    help="instead of the benchmark line: time and peak memory of the sweep workload at every context "
                         "length, with the T log T / T fits (one JSON object)")
    return ap.parse_args()


def get_spec(args, rank=0):
    from paper_2510_19875_b200 import workloads as wl

    spec = wl.SPECS[args.workload]
    if args.T:
        spec = spec.scaled(T=args.T)
    if rank:
        spec = spec.scaled(seed=spec.seed + 1000 * rank)
    return spec


def workload_config(spec, extra=None):
    cfg = {
        "workload": spec.name, "batch": spec.batch, "n_q_heads": spec.n_q_heads, "n_kv_heads": spec.n_kv_heads,
        "T": spec.T, "head_dim": spec.d, "block_q": spec.block, "block_k": spec.block, "k_top": spec.k_top,
        "causal": True, "seed": spec.seed,
        "structure": [n for n in ("sink", "local", "anchors", "needle") if getattr(spec, n)],
    }
    cfg.update(extra or {})
    return cfg


class ClockSampler:
    """nvidia-smi clocks and throttle reasons, sampled every 50 ms while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.lines, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._pump, daemon=True).start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])), mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except (OSError, KeyError, ValueError):
        return FALLBACK_HBM_GBS, "fallback"


def tensor_peak():
    """Measured dense bf16 throughput for a kernel timed inside a longer step (TFLOP/s)."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["bf16_tflops_sustained"]), "measured (sustained)"
    except (OSError, KeyError, ValueError):
        return FALLBACK_BF16_TFLOPS, "fallback (sustained)"


KERNEL_SOURCES = {
    "mask_tc_kernel": ("mask_tc.cu", "tc_common.cuh", "common.cuh"),
    "attn_tc_kernel": ("attn_tc.cu", "tc_common.cuh", "common.cuh"),
}


def kernel_source_hash(kernel: str) -> str:
    """Hash of the sources a kernel is built from; a stored ncu figure is only valid for the same hash."""
    import hashlib

    h = hashlib.sha256()
    for name in KERNEL_SOURCES[kernel]:
        with open(os.path.join(ROOT, "paper_2510_19875_b200", "csrc", name), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def ncu_traffic(kernel: str, spec):
    """DRAM bytes (read + write) per launch of `kernel` on this workload, from the committed ncu
    capture of the same workload at a smaller context length, scaled by T: the DRAM traffic of
    both kernels is their compulsory traffic (Q, K, V in, mask or output out, everything else is
    served by L2), which grows in proportion to T. None if there is no capture of this workload's
    shape or the kernel's sources changed since it was taken."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.json")
    try:
        with open(path) as fh:
            rec = json.load(fh)[kernel]
        if rec["source_hash"] != kernel_source_hash(kernel) or rec["workload"] != spec.name:
            return None
        return float(rec["dram_bytes_per_launch"]) * spec.T / float(rec["T"])
    except (OSError, KeyError, ValueError):
        return None


# The two SM units the tensor-core kernels lean on, measured on the device by the library's own
# probe (stream_probe_unit_rates) right before the timed steps: the bytes per clock two issuing
# warps bring from L2 into one SM's shared memory through TMA, and the clocks one tcgen05.mma of
# the mask kernel's shape takes. The bench line sets each kernel's traffic and instruction count against them.
TC_KERNELS = ("mask_tc_kernel", "attn_tc_kernel")


def rank_env():
    """(world size, rank, local rank) as torchrun exports them; (1, 0, 0) when run directly."""
    return (int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0")),
            int(os.environ.get("LOCAL_RANK", "0")))


def max_over_ranks(values, device):
    """Element-wise maximum over the ranks of a list of floats (the slowest rank sets the time)."""
    import torch
    import torch.distributed as dist

    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def job_value(world: int, units_per_rank: int, steps: int, total_ms: float) -> float:
    """Whole-job throughput: every rank processes `units_per_rank` per step (weak scaling)."""
    return world * units_per_rank * steps / (total_ms * 1e-3)


def oracle_sample_rate(spec, w, seconds: float):
    """Times the oracle (mask rows + attention rows, literal mode) on a seeded row sample sized for
    about `seconds` of wall time; returns (query-token-heads/s, threads, description)."""
    import numpy as np

    from oracle import stream_oracle as so

    p = so.OracleProblem(spec.batch, spec.n_q_heads, spec.n_kv_heads, spec.T, spec.d, spec.block, spec.block,
                         spec.k_top, True, spec.dtype)
    rng = np.random.default_rng(1234)
    threads = so.threads()

    def run(n):
        rows = np.sort(rng.choice(spec.n_rows, size=min(n, spec.n_rows), replace=False))
        t0 = time.perf_counter()
        res = so.build_mask_rows(p, w.q, w.k, rows)
        so.sparse_attention_rows(p, w.q, w.k, w.v, res["mask"], rows)
        return time.perf_counter() - t0, len(rows)

    t_probe, n_probe = run(2 * threads)
    n = int(max(2 * threads, min(spec.n_rows, seconds / max(t_probe, 1e-6) * n_probe)))
    t, n = run(n)
    return n * spec.block / t, threads, f"{n} seeded rows of {spec.n_rows} (mask + attention), {t:.1f} s wall"


def run_reference(args):
    """The oracle as the reference arm: each step is a bounded row sample of the same workload."""
    if rank_env()[1] != 0:
        return
    import numpy as np

    from oracle import stream_oracle as so
    from paper_2510_19875_b200 import workloads as wl

    spec = get_spec(args)
    w = wl.generate(spec)
    p = so.OracleProblem(spec.batch, spec.n_q_heads, spec.n_kv_heads, spec.T, spec.d, spec.block, spec.block,
                         spec.k_top, True, spec.dtype)
    threads = so.threads()
    rng = np.random.default_rng(1234)
    budget = 120.0 / max(1, args.steps + args.warmup)  # whole run within a few minutes

    def step(n):
        rows = np.sort(rng.choice(spec.n_rows, size=min(n, spec.n_rows), replace=False))
        t0 = time.perf_counter()
        res = so.build_mask_rows(p, w.q, w.k, rows)
        so.sparse_attention_rows(p, w.q, w.k, w.v, res["mask"], rows)
        return time.perf_counter() - t0

    t_probe = step(2 * threads)
    n = int(max(2 * threads, min(spec.n_rows, budget / max(t_probe, 1e-6) * 2 * threads)))
    for _ in range(args.warmup):
        step(n)
    times = [step(n) for _ in range(args.steps)]
    total = sum(times)
    value = n * spec.block * args.steps / total
    sample = f"{n} seeded rows of {spec.n_rows} per step (mask + attention)"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": workload_config(spec, {"sample": sample}),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2510_19875_b200 import stream as S
    from paper_2510_19875_b200 import workloads as wl

    world, rank, local = rank_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path for the library")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    spec = get_spec(args, rank)
    w = wl.generate(spec)
    qh, kh, vh = w.torch_tensors("cpu")
    q, k, v = qh.to(dev), kh.to(dev), vh.to(dev)
    kw = dict(block_q=spec.block, block_k=spec.block, k_top=spec.k_top)
    p = S.make_problem(q, k, impl=args.kernels, **kw)
    nqb = S.n_query_blocks(p)
    mask = torch.empty((spec.batch, spec.n_q_heads, nqb, spec.k_top), dtype=torch.int32, device=dev)
    out = torch.empty_like(q)
    ws = S.new_workspace(p, dev)
    stream = torch.cuda.current_stream()
    k_row = k_row_host = None
    if args.k_sparsity > 0:
        k_row_host = S.k_schedule(p, args.k_sparsity)
        k_row = k_row_host.to(dev)

    def build_mask():
        if k_row is None:
            S.stream_build_mask(p, q, k, mask, None, ws, ws.numel(), stream)
        else:
            S.stream_build_mask_var(p, q, k, k_row, mask, None, ws, ws.numel(), stream)

    def step():
        build_mask()
        S.stream_sparse_attention(p, q, k, v, mask, 0.0, out, stream)

    # the device's own unit rates (two short probe kernels, outside the timed region)
    unit_rates = None
    if rank == 0 and spec.dtype == "bf16" and args.kernels != "generic":
        unit_rates = S.probe_unit_rates(dev, stream)
    for _ in range(args.warmup):
        step()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    t_begin.record()
    for i in range(args.steps):
        ev[i][0].record()
        build_mask()
        ev[i][1].record()
        S.stream_sparse_attention(p, q, k, v, mask, 0.0, out, stream)
        ev[i][2].record()
    t_end.record()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    clocks = sampler.stop() if rank == 0 else None
    total_ms = t_begin.elapsed_time(t_end)
    mask_ms = statistics.mean(e[0].elapsed_time(e[1]) for e in ev)
    attn_ms = statistics.mean(e[1].elapsed_time(e[2]) for e in ev)
    stats = S.stream_read_stats(ws, stream)
    kept = int((mask >= 0).sum().item())

    # end to end through the host entry point: pinned host tensors in, mask + output back
    e2e = None
    if not args.no_e2e:
        qp, kp, vp = qh.pin_memory(), kh.pin_memory(), vh.pin_memory()
        mask_host = torch.empty(mask.shape, dtype=torch.int32).pin_memory()
        out_host = torch.empty(out.shape, dtype=out.dtype).pin_memory()
        del out
        ph = S.make_problem(qp, kp, impl=args.kernels, **kw)
        staging = torch.empty(S.stream_host_staging_bytes(ph), dtype=torch.uint8, device=dev)
        n_e2e = max(1, min(args.steps, 5))
        def run_host():
            if k_row_host is None:
                S.stream_run_host(ph, qp, kp, vp, mask_host, out_host, 0.0, staging, staging.numel(), stream)
            else:
                S.stream_run_host_var(ph, qp, kp, vp, k_row_host, mask_host, out_host, 0.0, staging, staging.numel(), stream)

        for _ in range(2):
            run_host()
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(n_e2e):
            run_host()
        b.record()
        torch.cuda.synchronize()
        e2e_ms = a.elapsed_time(b) / n_e2e
        assert torch.equal(mask_host, mask.cpu()), "host path produced a different mask"
        e2e = {"ms": e2e_ms, "steps": n_e2e,
               "h2d": qp.numel() * qp.element_size() + 2 * kp.numel() * kp.element_size(),
               "d2h": mask_host.numel() * 4 + out_host.numel() * out_host.element_size()}

    total_ms, mask_ms, attn_ms, e2e_ms = max_over_ranks([total_ms, mask_ms, attn_ms, e2e["ms"] if e2e else 0.0], dev)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    units = spec.batch * spec.n_q_heads * spec.T  # query-token-heads per rank per step
    esz = 2 if spec.dtype == "bf16" else 4
    S_tiles = int(stats.tiles_scored)
    tile_bytes = spec.block * spec.d * esz
    peak, peak_kind = hbm_peak()
    tc = spec.dtype == "bf16" and spec.d == 128 and spec.block == 64 and args.kernels != "generic"
    # algorithmic bytes per launch: every scored / kept tile counted as one fetch, Q in, result out
    kernels = {
        "stream_build_mask": {
            "kernel": "mask_tc_kernel" if tc and spec.k_top <= 32 else "mask_generic_kernel", "ms": mask_ms,
            "algorithmic_bytes": S_tiles * tile_bytes + units * spec.d * esz + spec.n_rows * spec.k_top * 4,
            "tiles_scored": S_tiles, "value": units / (mask_ms * 1e-3), "unit": UNIT,
            "tensor_tflops": S_tiles * 2.0 * spec.block * spec.block * spec.d / (mask_ms * 1e-3) / 1e12},
        "stream_sparse_attention": {
            "kernel": "attn_tc_kernel" if tc else "attn_generic_kernel", "ms": attn_ms,
            "algorithmic_bytes": kept * 2 * tile_bytes + 2 * units * spec.d * esz, "kept_blocks": kept,
            "tensor_tflops": kept * 4.0 * spec.block * spec.block * spec.d / (attn_ms * 1e-3) / 1e12},
    }
    for rec in kernels.values():
        rec["algorithmic_gbs"] = rec["algorithmic_bytes"] / (rec["ms"] * 1e-3) / 1e9
        rec["frac_of_hbm_peak"] = rec["algorithmic_gbs"] / peak
    dominant = max(kernels, key=lambda n: kernels[n]["ms"])
    dom = kernels[dominant]
    tpeak, tpeak_kind = tensor_peak()
    n_sm = torch.cuda.get_device_properties(dev).multi_processor_count
    sm_mhz = (clocks or {}).get("sm_mhz") or 1965.0
    # Which roof binds the dominant kernel: the time its tile FLOPs need at the measured tensor
    # peak against the time its compulsory DRAM traffic (every input read once, the result written
    # once) needs at the measured HBM peak; the larger one is the bound and frac = that time / the
    # measured time. The gathers of key tiles are served by L2 (compare `traffic`), which is why
    # the HBM figure on algorithmic bytes is given separately and is not a fraction of a bound.
    flops = dom["tensor_tflops"] * 1e12 * dom["ms"] * 1e-3
    compulsory = (units * spec.d * esz + spec.batch * spec.n_kv_heads * spec.T * spec.d * esz + spec.n_rows * spec.k_top * 4
                  if dominant == "stream_build_mask" else
                  2 * units * spec.d * esz + 2 * spec.batch * spec.n_kv_heads * spec.T * spec.d * esz + spec.n_rows * spec.k_top * 4)
    t_tensor_ms = flops / (tpeak * 1e12) * 1e3 if tc else 0.0
    t_hbm_ms = compulsory / (peak * 1e9) * 1e3
    traffic = ncu_traffic(dom["kernel"], spec) if dom["kernel"] in KERNEL_SOURCES and k_row is None else None
    if tc and t_tensor_ms >= t_hbm_ms:
        roof = {"bound": "tensor", "achieved": dom["tensor_tflops"], "peak": tpeak, "unit": "TFLOP/s",
                "frac": dom["tensor_tflops"] / tpeak, "peak_kind": f"of {tpeak_kind}"}
    elif tc or spec.dtype == "bf16":
        roof = {"bound": "hbm", "achieved": compulsory / (dom["ms"] * 1e-3) / 1e9, "peak": peak, "unit": "GB/s",
                "frac": t_hbm_ms / dom["ms"], "peak_kind": f"of {peak_kind}"}
    else:  # the generic kernels: plain fp32 FMA arithmetic
        alu_peak = n_sm * 128 * 2 * 1.965e9 / 1e12  # SMs x FMA lanes x 2 FLOP x max SM clock
        roof = {"bound": "alu", "achieved": dom["tensor_tflops"], "peak": alu_peak, "unit": "TFLOP/s",
                "frac": dom["tensor_tflops"] / alu_peak, "peak_kind": "SMs x 128 FMA lanes x 2 x 1.965 GHz"}
    roof.update({
        "kernel": dom["kernel"], "entry_point": dominant, "traffic": traffic,
        "traffic_kind": "ncu dram bytes of a capture at a smaller T of the same workload, scaled by T (compulsory traffic)",
        "share_of_step": dom["ms"] / (mask_ms + attn_ms),
        "bound_times_ms": {"tensor": t_tensor_ms, "hbm_compulsory": t_hbm_ms, "measured": dom["ms"]},
        # the metric's own accounting: every scored (kept) tile counted as one fetch from memory.
        # On this GPU those fetches are L2 hits, so this can exceed 1 and is not the binding roof.
        "hbm_algorithmic": {"achieved": dom["algorithmic_gbs"], "peak": peak, "unit": "GB/s",
                            "frac": dom["algorithmic_gbs"] / peak, "peak_kind": f"of {peak_kind}",
                            "algorithmic_bytes": dom["algorithmic_bytes"],
                            "frac_of_8TBs_nominal": dom["algorithmic_gbs"] / 8000.0,
                            "note": "served by L2: DRAM carries only `traffic`"},
    })
    if dom["kernel"] in TC_KERNELS and unit_rates is not None:
        cycles = dom["ms"] * 1e-3 * sm_mhz * 1e6  # per SM, at the sampled clock
        if dominant == "stream_build_mask":
            gathered = int(stats.tiles_fetched) * tile_bytes          # counted by the kernel
            mma_cycles = S_tiles / 2 * 8 * unit_rates.mma_cycles_m128n64 / n_sm   # chains of two tiles, eight MMAs each
        else:
            gathered = kept * 2 * tile_bytes + units * spec.d * esz   # K and V tile per kept block, Q once
            mma_cycles = None
        per_clk = gathered / n_sm / cycles
        roof["unit_rates"] = {
            "sm_mhz": sm_mhz, "kind": "measured by stream_probe_unit_rates on this device before the timed steps",
            "tma_bytes_per_clk_per_sm": unit_rates.tma_bytes_per_clk, "mma_m128n64k16_cycles": unit_rates.mma_cycles_m128n64,
            "tma_gather": {"bytes": gathered, "achieved": per_clk, "peak": unit_rates.tma_bytes_per_clk,
                           "unit": "B/clk/SM", "frac": per_clk / unit_rates.tma_bytes_per_clk},
        }
        if mma_cycles is not None:
            roof["unit_rates"]["mma_issue"] = {"cycles_needed": mma_cycles, "cycles_measured": cycles, "frac": mma_cycles / cycles}
    line = {
        "metric": METRIC, "value": job_value(world, units, args.steps, total_ms), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": spec.dtype, "data": "synthetic",
        "config": workload_config(spec, {"l2": "inputs larger than L2 (Q+K+V %.0f MiB per step)" % (
            (q.numel() + 2 * k.numel()) * esz / 2**20), "kernels": args.kernels, "per_rank": "one independent layer each",
            **({"k_schedule": {"effective_sparsity": args.k_sparsity, "k_min": int(k_row.min()), "k_max": int(k_row.max()),
                               "k_mean": float(k_row.float().mean())}} if k_row is not None else {})}),
        "mask_build": kernels["stream_build_mask"], "sparse_attention": kernels["stream_sparse_attention"],
        "roofline": roof,
        "clocks": clocks,
        "gpu_launches": 2 * args.steps,
    }
    if e2e:
        line["e2e"] = {"value": world * units / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms,
                       "h2d_bytes_per_step": e2e["h2d"], "d2h_bytes_per_step": e2e["d2h"], "steps": e2e["steps"]}
    del q, k, v, mask
    if world == 1 and not args.no_sweep:
        # the scaling sweep's three shortest context lengths (the full sweep is `--sweep`): time and
        # peak device memory against T, so that "memory linear in T" has a record in this line
        rows = sweep_rows(wl.SWEEP_T[:3], dev)
        line["sweep"] = {"rows": [{k2: r[k2] for k2 in ("T", "levels", "mask_ms", "attention_ms", "peak_device_bytes")} for r in rows],
                         **sweep_fits(rows)}
        # and the two small workloads (a single fp32 head; a 16k-token GQA layer), device-resident, best of 3
        small = {}
        for name in ("single_head_fp32", "gqa_layer_16k"):
            if name == spec.name:
                continue
            sp = wl.SPECS[name]
            ws_ = wl.generate(sp)
            q2, k2, v2 = ws_.torch_tensors(dev)
            p2 = S.make_problem(q2, k2, block_q=sp.block, block_k=sp.block, k_top=sp.k_top, impl=args.kernels)
            m2 = torch.empty((sp.batch, sp.n_q_heads, S.n_query_blocks(p2), sp.k_top), dtype=torch.int32, device=dev)
            o2 = torch.empty_like(q2)
            w2 = S.new_workspace(p2, dev)
            best = [float("inf"), float("inf")]
            for it in range(5):
                e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
                e0.record()
                S.stream_build_mask(p2, q2, k2, m2, None, w2, w2.numel(), stream)
                e1.record()
                S.stream_sparse_attention(p2, q2, k2, v2, m2, 0.0, o2, stream)
                e2.record()
                torch.cuda.synchronize()
                if it >= 2:
                    best = [min(best[0], e0.elapsed_time(e1)), min(best[1], e1.elapsed_time(e2))]
            small[name] = {"mask_ms": best[0], "attention_ms": best[1], "T": sp.T, "dtype": sp.dtype,
                           "value": sp.batch * sp.n_q_heads * sp.T / ((best[0] + best[1]) * 1e-3), "unit": UNIT}
            del q2, k2, v2, m2, o2
        line["other_workloads"] = small
    if not args.no_cpu_baseline:
        rate, threads, sample = oracle_sample_rate(spec, w, args.cpu_seconds)
        line["cpu_baseline"] = {"value": rate, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def fit_r2(x, y, through_origin):
    """Least-squares line y ~ a x (+ b); returns (a, b, R^2)."""
    import numpy as np

    x, y = np.asarray(x, float), np.asarray(y, float)
    if through_origin:
        a, b = float((x * y).sum() / (x * x).sum()), 0.0
    else:
        a, b = (float(v) for v in np.polyfit(x, y, 1))
    ss_res, ss_tot = float(((y - (a * x + b)) ** 2).sum()), float(((y - y.mean()) ** 2).sum())
    return a, b, 1.0 - ss_res / ss_tot


def sweep_rows(Ts, dev):
    """Time of both kernels and peak device memory of the sweep workload at each context length in Ts."""
    import math

    import torch

    from paper_2510_19875_b200 import stream as S
    from paper_2510_19875_b200 import workloads as wl

    rows = []
    for T in Ts:
        spec = wl.SPECS["sweep"].scaled(T=T)
        w = wl.generate(spec)
        torch.cuda.empty_cache()
        torch.cuda.reset_peak_memory_stats()
        base = torch.cuda.memory_allocated()
        q, k, v = w.torch_tensors(dev)
        kw = dict(block_q=spec.block, block_k=spec.block, k_top=spec.k_top)
        p = S.make_problem(q, k, **kw)
        mask = torch.empty((spec.batch, spec.n_q_heads, S.n_query_blocks(p), spec.k_top), dtype=torch.int32, device=dev)
        out = torch.empty_like(q)
        ws = S.new_workspace(p, dev)
        stream = torch.cuda.current_stream()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        best = [float("inf"), float("inf")]
        for it in range(5):
            ev[0].record()
            S.stream_build_mask(p, q, k, mask, None, ws, ws.numel(), stream)
            ev[1].record()
            S.stream_sparse_attention(p, q, k, v, mask, 0.0, out, stream)
            ev[2].record()
            torch.cuda.synchronize()
            if it >= 2:
                best = [min(best[0], ev[0].elapsed_time(ev[1])), min(best[1], ev[1].elapsed_time(ev[2]))]
        tiles = int(S.stream_read_stats(ws, stream).tiles_scored)
        n_kb = -(-T // spec.block)
        levels = max(1, math.ceil(math.log2(max(1, -(-n_kb // spec.k_top))))) if n_kb > 1 else 0
        rows.append({"T": T, "levels": levels, "mask_ms": best[0], "attention_ms": best[1], "tiles_scored": tiles,
                     "peak_device_bytes": int(torch.cuda.max_memory_allocated() - base),
                     "input_output_bytes": int((2 * q.numel() + 2 * k.numel()) * q.element_size() + mask.numel() * 4),
                     "workspace_bytes": int(ws.numel())})
        del q, k, v, out, mask, w
    return rows


def sweep_fits(rows):
    Ts = [r["T"] for r in rows]
    a, _, r2_time = fit_r2([r["T"] * (r["levels"] + 1) for r in rows], [r["mask_ms"] for r in rows], True)
    a_lin, _, r2_lin = fit_r2(Ts, [r["mask_ms"] for r in rows], True)
    m_a, m_b, r2_mem = fit_r2(Ts, [r["peak_device_bytes"] for r in rows], False)
    return {"fit_mask_time_vs_T_levels": {"ms_per_token_level": a, "r2": r2_time},
            "fit_mask_time_vs_T": {"ms_per_token": a_lin, "r2": r2_lin},
            "fit_peak_memory_vs_T": {"bytes_per_token": m_a, "offset_bytes": m_b, "r2": r2_mem}}


def run_sweep(args):
    """Scaling of the path with the context length (the paper's complexity ablation, App. A.3): time of
    both kernels and peak device memory at every T of the sweep workload, and the fits time ~ T (L + 1)
    (L = levels of the hierarchy, about log2(T / (block k))) and memory ~ T."""
    import torch

    from paper_2510_19875_b200 import workloads as wl

    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    rows = sweep_rows(wl.SWEEP_T, dev)
    print(json.dumps({"workload": "sweep", "rows": rows, **sweep_fits(rows)}))


def run_k_list(args):
    """The several-k mask build (the search over k of Section 3 wants the masks of one input for
    more than one k): one call that shares tile scores between the k, against the same call with
    the small workspace (one launch per k, nothing shared)."""
    import torch

    from paper_2510_19875_b200 import stream as S
    from paper_2510_19875_b200 import workloads as wl

    ks = [int(x) for x in args.k_list.split(",")]
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    spec = get_spec(args, 0)
    w = wl.generate(spec)
    q, k, _ = w.torch_tensors(dev)
    out = {"workload": spec.name, "T": spec.T, "k_list": ks, "kernels": args.kernels}
    for name, share in (("shared", True), ("per_k", False)):
        best, res = float("inf"), None
        for it in range(args.warmup + args.steps):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            res = S.build_masks(q, k, ks, block_q=spec.block, block_k=spec.block, impl=args.kernels, share=share)
            b.record()
            torch.cuda.synchronize()
            if it >= args.warmup:
                best = min(best, a.elapsed_time(b))
        out[name] = {"ms": best, "tiles_scored": int(res.stats().tiles_scored), "workspace_bytes": int(res.workspace.numel())}
    print(json.dumps(out))


def run_per_token(args):
    """The per-token mask build (block_q = 1, block_k = the workload's block): one step = one
    stream_build_mask call on the workload's Q and K (masks only: the attention pass for
    per-token masks runs on the generic kernel and is not part of this line)."""
    import torch

    from paper_2510_19875_b200 import stream as S
    from paper_2510_19875_b200 import workloads as wl

    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    spec = get_spec(args, 0)
    w = wl.generate(spec, with_v=False)
    q, k, _ = w.torch_tensors(dev)
    p = S.make_problem(q, k, block_q=1, block_k=spec.block, k_top=spec.k_top, impl=args.kernels)
    mask = torch.empty((spec.batch, spec.n_q_heads, spec.T, spec.k_top), dtype=torch.int32, device=dev)
    ws = S.new_workspace(p, dev)
    stream = torch.cuda.current_stream()
    for _ in range(args.warmup):
        S.stream_build_mask(p, q, k, mask, None, ws, ws.numel(), stream)
    sampler = ClockSampler(0)
    sampler.start()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    a.record()
    for _ in range(args.steps):
        S.stream_build_mask(p, q, k, mask, None, ws, ws.numel(), stream)
    b.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = a.elapsed_time(b) / args.steps
    st = S.stream_read_stats(ws, stream)
    units = spec.batch * spec.n_q_heads * spec.T
    esz = 2 if spec.dtype == "bf16" else 4
    tile_flops = 2.0 * 64 * 64 * spec.d
    tpeak, tpeak_kind = tensor_peak()
    peak, peak_kind = hbm_peak()
    products = int(st.tile_products)
    on_tensor = products > 0
    achieved = products * tile_flops / (ms * 1e-3) / 1e12
    compulsory = units * spec.d * esz + spec.batch * spec.n_kv_heads * spec.T * spec.d * esz + units * spec.k_top * 4
    line = {
        "metric": METRIC, "value": units / (ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": spec.dtype,
        "data": "synthetic",
        "config": workload_config(spec, {"block_q": 1, "kernels": args.kernels, "step": "per-token mask build only",
                                         "l2": "inputs larger than L2" if (q.numel() + k.numel()) * esz > 126e6 else "inputs fit L2"}),
        "mask_build": {"kernel": "mask_tok_kernel" if on_tensor else "mask_generic_kernel", "ms": ms,
                       "tiles_scored": int(st.tiles_scored), "tile_products": products,
                       "useful_fraction_of_products": (int(st.tiles_scored) / 64.0) / products if products else None},
        "roofline": {"bound": "tensor", "kernel": "mask_tok_kernel", "entry_point": "stream_build_mask", "achieved": achieved,
                     "peak": tpeak, "unit": "TFLOP/s", "frac": achieved / tpeak, "peak_kind": f"of {tpeak_kind}", "traffic": None,
                     "flops": "tile products the kernel computed (every fetched key tile x 128 tokens) x 2 x 64 x 64 x d",
                     "bound_times_ms": {"tensor": products * tile_flops / (tpeak * 1e12) * 1e3,
                                        "hbm_compulsory": compulsory / (peak * 1e9) * 1e3, "measured": ms}} if on_tensor else None,
        "clocks": clocks, "gpu_launches": args.steps, "e2e": None,
    }
    if not args.no_cpu_baseline:
        import numpy as np

        from oracle import stream_oracle as so

        op = so.OracleProblem(spec.batch, spec.n_q_heads, spec.n_kv_heads, spec.T, spec.d, 1, spec.block, spec.k_top, True, spec.dtype)
        rng = np.random.default_rng(1234)
        n = 64 * so.threads()
        t_cpu = 0.0
        while True:
            rows = np.sort(rng.choice(units, size=min(n, units), replace=False))
            t0 = time.perf_counter()
            so.build_mask_rows(op, w.q, w.k, rows)
            t_cpu = time.perf_counter() - t0
            if t_cpu > args.cpu_seconds / 3 or n >= units:
                break
            n = int(n * max(2.0, args.cpu_seconds / max(t_cpu, 1e-3) * 0.7))
        line["cpu_baseline"] = {"value": len(rows) / t_cpu, "unit": UNIT, "cores": so.threads(), "kind": "oracle",
                                "sample": f"{len(rows)} seeded token rows of {units} (mask only), {t_cpu:.1f} s wall"}
    print(json.dumps(line))


def run_extras(args):
    """The kernels around the mask: vertical scores + kurtosis (binary and score-weighted), mask
    subtraction (k against k / 2), and the several-k build (k / 4, k / 2, k in one call against the
    k build alone). The first two are scans of the masks: bytes moved / time against the HBM peak."""
    import torch

    from paper_2510_19875_b200 import stream as S
    from paper_2510_19875_b200 import workloads as wl

    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    spec = get_spec(args, 0)
    w = wl.generate(spec, with_v=False)
    q, k, _ = w.torch_tensors(dev)
    kw = dict(block_q=spec.block, block_k=spec.block)
    peak, peak_kind = hbm_peak()

    def best_ms(fn):
        best = float("inf")
        for it in range(args.warmup + args.steps):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            fn()
            b.record()
            torch.cuda.synchronize()
            if it >= args.warmup:
                best = min(best, a.elapsed_time(b))
        return best

    big = S.build_mask(q, k, k_top=spec.k_top, want_scores=True, **kw)
    small = S.build_mask(q, k, k_top=max(1, spec.k_top // 2), **kw)
    torch.cuda.synchronize()
    p = S.make_problem(q, k, k_top=spec.k_top, **kw)
    n_kb = -(-spec.T // spec.block)
    rows = spec.n_rows
    mask_bytes = rows * spec.k_top * 4
    out = {"workload": spec.name, "T": spec.T, "k_top": spec.k_top, "rows": rows, "hbm_peak_gbs": peak, "peak_kind": peak_kind}

    vert = torch.empty((spec.batch, spec.n_q_heads, n_kb), dtype=torch.float32, device=dev)
    kurt = torch.empty((spec.batch, spec.n_q_heads), dtype=torch.float32, device=dev)
    ws = S.new_workspace(p, dev)
    for name, sc in (("vertical_binary", None), ("vertical_weighted", big.scores)):
        ms = best_ms(lambda: S.stream_vertical_scores(p, big.mask, sc, vert, kurt, ws, ws.numel()))
        nbytes = mask_bytes * (2 if sc is not None else 1) + vert.numel() * 4
        out[name] = {"ms": ms, "bytes": nbytes, "gbs": nbytes / (ms * 1e-3) / 1e9, "frac_of_hbm_peak": nbytes / (ms * 1e-3) / 1e9 / peak}

    diff = torch.empty_like(big.mask)
    dsc = torch.empty_like(big.scores)
    ms = best_ms(lambda: S.stream_mask_difference(rows, spec.k_top, big.mask, big.scores, small.mask.shape[-1], small.mask, diff, dsc))
    nbytes = mask_bytes * 4 + small.mask.numel() * 4  # mask and scores of a in, of the difference out; mask b in
    out["mask_difference"] = {"ms": ms, "bytes": nbytes, "gbs": nbytes / (ms * 1e-3) / 1e9, "frac_of_hbm_peak": nbytes / (ms * 1e-3) / 1e9 / peak}

    ks = sorted({max(1, spec.k_top // 4), max(1, spec.k_top // 2), spec.k_top})
    one = best_ms(lambda: S.build_mask(q, k, k_top=spec.k_top, impl=args.kernels, **kw))
    res = None

    def multi():
        nonlocal res
        res = S.build_masks(q, k, ks, impl=args.kernels, **kw)
    shared = best_ms(multi)
    out["several_k"] = {"k_list": ks, "ms": shared, "ms_largest_k_alone": one, "ratio": shared / one,
                        "tiles_scored": int(res.stats().tiles_scored)}
    print(json.dumps(out))


def main():
    args = parse_args()
    if args.extras:
        run_extras(args)
        return
    if args.block_q == 1:
        run_per_token(args)
        return
    if args.k_list:
        run_k_list(args)
        return
    if args.sweep:
        run_sweep(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

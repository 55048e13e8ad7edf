#!/usr/bin/env python
"""Benchmark of LoSA's attention hot path on B200.

One "step" is one pass of the whole path over one synthetic attention layer:

    losa_block_mass(q0, k0) -> losa_select(mass, tau)           (one-time construction)
    losa_sparse_attn(q_t, k_t, v_t, CSR) for t = 1..draws        (frozen pattern, later steps)
    losa_attn(q_1, k_1, v_1)                                     (own dense forward, for the ratio)
    losa_attn_mass(q_1, k_1, v_1)                                (construction step as one kernel)

The headline value is the effective TFLOP/s of the block-sparse forward, counting the flops of
the retained blocks only.  Everything is timed with CUDA events on the launching stream.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload wan] [--draws 10]
    python bench.py --impl reference ...      # the fp64 CPU oracle on a bounded sample

Under torchrun every rank runs the same layer shape on its own seeds (weak scaling; the path has
no exchange step, so there is no data-path collective) and rank 0 prints one JSON line.  With
`--shard heads` the ranks split the heads of ONE layer instead (strong scaling, still no collective:
every head is independent and a CSR row belongs to one head).
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

from paper_2608_12032_b200 import inputs  # noqa: E402

METRIC = "block_sparse_attn_effective_tflops"
UNIT = "TFLOP/s"
NOMINAL_BF16_TFLOPS = 2250.0
# dram__bytes_read.sum + dram__bytes_write.sum of one sparse-forward launch, from an ncu capture of
# the same kernel on the same workload (a profiler run: not re-measured by this script, which never
# runs under a profiler); None where no capture was taken
NCU_DRAM_BYTES_PER_LAUNCH = {"wan": 0.303640e9 + 0.082585e9}
NCU_TRAFFIC_SOURCE = "ncu capture of the sparse forward at the Wan2.1 shape (dram__bytes_read.sum + dram__bytes_write.sum)"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def merge_kernel_runs(wl) -> bool:
    """Whether the attention-only calls launch their merge kernel for this shape: the library says how
    many work slots a call occupies; work items are pairs of 128-row query tiles per head, and the
    items of a last, partly filled wave are cut into parts (at most 8, at most one per key block)."""
    from paper_2608_12032_b200 import binding
    prob = binding.Problem(wl.B, wl.H, wl.N, wl.D, wl.R, wl.C, wl.H * wl.N * wl.D, wl.N * wl.D, wl.D, 0.0)
    ctas = binding.losa_work_slots(binding.LOSA_OP_SPARSE_ATTN, prob)
    n_work = wl.B * wl.H * ((-(-wl.N // 128) + 1) // 2)
    rest = n_work if n_work < ctas else n_work % ctas
    parts = min(ctas // rest, 8, -(-wl.N // wl.C)) if rest else 1
    return parts >= 2


def launches_per_step(wl, draws: int) -> int:
    """Kernels of the library launched by one step.  Every attention-shaped call launches its kernel
    and the fallback kernel behind it (which returns at once when no row outgrew its reference): the
    mass pass 2; select 3; every sparse call also its tile-list pre-pass, plus the merge kernel when the
    last wave is cut into parts; the dense call the same without the pre-pass; the fused step 2."""
    merge = int(merge_kernel_runs(wl))
    return 2 + 3 + draws * (3 + merge) + (2 + merge) + 2


def cpu_model() -> str:
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.lower().startswith("model name"):
                    return line.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="losa", choices=["losa", "reference"])
    ap.add_argument("--workload", default="wan", choices=sorted(inputs.WORKLOADS))
    ap.add_argument("--draws", type=int, default=10, help="reuse draws per step")
    ap.add_argument("--tau", type=float, default=None)
    ap.add_argument("--cpu-seconds", type=float, default=12.0, help="budget of the CPU-baseline sample")
    ap.add_argument("--shard", default="replicas", choices=["replicas", "heads"],
                    help="N > 1: every rank its own layer (weak scaling), or the heads of one layer split "
                         "across the ranks (strong scaling); no collective inside the path either way")
    ap.add_argument("--batched-layers", type=int, default=0,
                    help="also time losa_sparse_attn_batched over this many layers against the single calls")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    return ap.parse_args()


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        d["_source"] = "measured"
        return d
    d = dict(FALLBACK_PEAKS)
    d["_source"] = "fallback"
    return d


def retained_flops(wl, offsets: np.ndarray, kv_idx: np.ndarray) -> float:
    """4 * d * sum over retained (query block, key block) pairs of |B_i| * |B_j| (valid tokens)."""
    nQb, nKb = wl.nQb, wl.nKb
    qsz = np.full(nQb, wl.R, dtype=np.int64)
    qsz[-1] = wl.N - (nQb - 1) * wl.R
    ksz = np.full(nKb, wl.C, dtype=np.int64)
    ksz[-1] = wl.N - (nKb - 1) * wl.C
    counts = np.diff(offsets.astype(np.int64))
    row_q = np.tile(qsz, wl.B * wl.H)
    per_entry_q = np.repeat(row_q, counts)
    return 4.0 * wl.D * float((per_entry_q * ksz[kv_idx[: offsets[-1]]]).sum())


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int):
        self.samples, self.power, self.reasons = [], [], set()
        self.max_mhz = None
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
        names = {
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    self.power.append(nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0)
                except Exception:
                    pass
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.01)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        return {
            "sm_mhz": statistics.median(self.samples) if self.samples else None,
            "sm_max_mhz": self.max_mhz,
            "reasons": sorted(self.reasons),
            "samples": len(self.samples),
            "sm_min_mhz": min(self.samples) if self.samples else None,
            "power_w": statistics.median(self.power) if self.power else None,
        }


def max_over_ranks(values, dist, device):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    t = torch.tensor(values, dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.cpu()]


def sum_over_ranks(value: float, dist, device) -> float:
    """Sum of one float over all ranks (identity without a process group)."""
    t = torch.tensor([value], dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.cpu()[0])


def aggregate_tflops(flops_per_call: float, calls: int, slowest_rank_ms: float, world: int) -> float:
    """Whole-job throughput: every rank does `calls` launches of `flops_per_call`; the job takes as
    long as its slowest rank (weak scaling, no exchange between ranks)."""
    return world * flops_per_call * calls / (slowest_rank_ms * 1e-3) / 1e12


def cpu_baseline(wl, q, k, v, offsets, kv_idx, seconds: float, gpu_mass=None, tau=None):
    """The oracle, as it stands, on a bounded sample of query blocks: its sparse attention (Eq. 4)
    is the baseline value; its dense attention, block mass and selection are timed beside it on a
    few blocks, and the GPU's pattern is checked against the oracle's rule on the GPU's own masses."""
    from oracle import losa_oracle as orc

    qn, kn, vn = (t.float().numpy() for t in (q, k, v))
    rows = wl.rows
    rng = np.random.default_rng(0)
    order = rng.permutation(rows)
    nQb = wl.nQb
    done, flops, t0 = 0, 0.0, time.perf_counter()
    chunk = max(1, orc.threads() // 16)
    ksz = np.full(wl.nKb, wl.C, dtype=np.int64)
    ksz[-1] = wl.N - (wl.nKb - 1) * wl.C
    while done < rows:
        ids = np.sort(order[done:done + chunk]).astype(np.int32)
        orc.sparse_attn(qn, kn, vn, wl.R, wl.C, offsets, kv_idx, row_ids=ids)
        for r in ids:
            i = int(r) % nQb
            qrows = min(wl.R, wl.N - i * wl.R)
            flops += 4.0 * wl.D * qrows * float(ksz[kv_idx[offsets[r]:offsets[r + 1]]].sum())
        done += len(ids)
        if time.perf_counter() - t0 >= seconds:
            break
    dt = time.perf_counter() - t0
    out = {
        "value": flops / dt / 1e12,
        "unit": UNIT,
        "cores": orc.threads(),
        "cpu": cpu_model(),
        "kind": "oracle",
        "sample": f"fp64 oracle sparse attention on {done} of {rows} query blocks "
                  f"(random sample, seed 0) of the {wl.name} workload in {dt:.1f} s",
        "seconds": dt,
        "blocks": done,
    }
    # the other steps, each on a handful of blocks: seconds per query block and per full layer
    few = np.sort(order[: max(2, min(8, orc.threads() // 4))]).astype(np.int32)
    per_block = {"sparse_attn": dt / max(done, 1)}
    t0 = time.perf_counter()
    mass_few = orc.block_mass(qn, kn, wl.R, wl.C, row_ids=few)
    per_block["block_mass"] = (time.perf_counter() - t0) / len(few)
    counts = np.ones(rows, dtype=np.int64)
    counts[few] = wl.nKb
    doff = np.zeros(rows + 1, dtype=np.int64)
    np.cumsum(counts, out=doff[1:])
    didx = np.zeros(doff[-1], dtype=np.int32)
    for r in few:
        didx[doff[r]:doff[r + 1]] = np.arange(wl.nKb)
    t0 = time.perf_counter()
    orc.sparse_attn(qn, kn, vn, wl.R, wl.C, doff.astype(np.int32), didx, row_ids=few)
    per_block["dense_attn"] = (time.perf_counter() - t0) / len(few)
    out["oracle_seconds_per_query_block"] = per_block
    out["oracle_seconds_per_layer_extrapolated"] = {k_: v_ * rows for k_, v_ in per_block.items()}
    if gpu_mass is not None:
        # selection on every row of the GPU's own masses: oracle seconds, CSR equality, near-tau rows
        t0 = time.perf_counter()
        sel = orc.select(gpu_mass.astype(np.float64), tau)
        out["oracle_seconds_per_layer_extrapolated"]["select"] = time.perf_counter() - t0
        dist = sel.boundary_distance()
        ref_off = sel.offsets
        same = bool(np.array_equal(ref_off, offsets)) and bool(np.array_equal(sel.kv_idx, kv_idx[: offsets[-1]]))
        mism = 0
        if not same:
            for r in range(rows):
                a = kv_idx[offsets[r]:offsets[r + 1]]
                b = sel.kv_idx[ref_off[r]:ref_off[r + 1]]
                if a.shape != b.shape or not np.array_equal(a, b):
                    mism += 1
        out["select_check"] = {
            "rows": int(rows), "csr_equals_oracle_rule_on_gpu_masses": same, "rows_that_differ": int(mism),
            "rows_within_1e-6_of_tau": int((dist < 1e-6).sum()),
            "min_distance_to_tau": float(dist.min()),
        }
        del mass_few
    return out


def run_reference(args, wl, rank, world):
    """Reference arm: the fp64 CPU oracle, timed on this machine's host cores (rank 0 only)."""
    if rank != 0:
        return
    from oracle import losa_oracle as orc

    tau = wl.tau if args.tau is None else args.tau
    q, k, v = inputs.make_qkv(wl, 0)
    qn, kn, vn = (t.float().numpy() for t in (q, k, v))
    # the pattern of a bounded sample of query blocks, from the oracle's own masses
    per_step = max(2, min(32, orc.threads()))
    rng = np.random.default_rng(0)
    total = args.warmup + args.steps
    ids_all = rng.choice(wl.rows, size=min(wl.rows, per_step * total), replace=False).astype(np.int32)
    times, flops = [], []
    ksz = np.full(wl.nKb, wl.C, dtype=np.int64)
    ksz[-1] = wl.N - (wl.nKb - 1) * wl.C
    for s in range(total):
        ids = np.sort(ids_all[s * per_step:(s + 1) * per_step])
        if ids.size == 0:
            ids = np.sort(ids_all[:per_step])
        t0 = time.perf_counter()
        mass = orc.block_mass(qn, kn, wl.R, wl.C, row_ids=ids)
        sel = orc.select(mass, tau)
        # CSR over all rows with only the sampled rows populated
        counts = np.ones(wl.rows, dtype=np.int64)
        counts[ids] = sel.count
        off = np.zeros(wl.rows + 1, dtype=np.int64)
        np.cumsum(counts, out=off[1:])
        idx = np.zeros(off[-1], dtype=np.int32)
        for n, r in enumerate(ids):
            idx[off[r]:off[r + 1]] = sel.kept[n, : sel.count[n]]
        t1 = time.perf_counter()
        orc.sparse_attn(qn, kn, vn, wl.R, wl.C, off.astype(np.int32), idx, row_ids=ids)
        t2 = time.perf_counter()
        f = 0.0
        for n, r in enumerate(ids):
            qrows = min(wl.R, wl.N - (int(r) % wl.nQb) * wl.R)
            f += 4.0 * wl.D * qrows * float(ksz[sel.kept[n, : sel.count[n]]].sum())
        if s >= args.warmup:
            times.append((t2 - t0, t2 - t1))
            flops.append(f)
    sparse_s = sum(t[1] for t in times)
    value = sum(flops) / sparse_s / 1e12
    line = {
        "impl": "reference",
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * sum(t[0] for t in times) / len(times),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": wl.name, "tau": tau, "sample_blocks_per_step": per_step,
                   "note": "each step = oracle mass + select + sparse attention on a sample of query blocks"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": orc.threads(), "kind": "oracle",
                         "sample": f"{per_step} random query blocks of {wl.rows} per step"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def main():
    args = parse_args()
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    wl = inputs.WORKLOADS[args.workload]

    if args.impl == "reference":
        run_reference(args, wl, rank, world)
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    import paper_2608_12032_b200 as losa

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=dev)

    tau = wl.tau if args.tau is None else args.tau
    shard_heads = args.shard == "heads" and world > 1
    # replicas: rank r draws its own layer; heads: every rank draws the same layer and keeps its heads
    base_seed = 0 if shard_heads else 1000 * rank
    peaks = load_peaks()

    # ---- inputs: step-0 tensors and the reuse draws, resident in HBM before timing starts
    base = inputs.make_base_fp32(wl, base_seed)
    q0, k0, v0 = (t.bfloat16() for t in base)
    host_draws = [inputs.make_reuse_draw(wl, base_seed + t, base=base) for t in range(1, args.draws + 1)]
    del base
    full_heads = wl.H
    if shard_heads:
        # heads [h0, h1) of the layer: every (batch, head) is independent in all four calls and a CSR
        # row belongs to one head, so the ranks exchange nothing inside the path
        from paper_2608_12032_b200 import sharding

        h0, h1 = sharding.head_range(wl.H, rank, world)
        q0, k0, v0 = (sharding.shard_heads(t, rank, world).contiguous() for t in (q0, k0, v0))
        host_draws = [tuple(sharding.shard_heads(t, rank, world).contiguous() for t in d) for d in host_draws]
        wl = dataclasses.replace(wl, H=h1 - h0)
    q0d, k0d = q0.to(dev), k0.to(dev)
    draws = [tuple(t.to(dev) for t in d) for d in host_draws]

    prob = losa.make_problem(q0d, wl.R, wl.C)
    rows, nKb = wl.rows, wl.nKb
    ws_mass = torch.empty(losa.losa_workspace_bytes(0, prob), dtype=torch.uint8, device=dev)
    mass = torch.empty((wl.B, wl.H, wl.nQb, nKb), dtype=torch.float32, device=dev)
    offsets = torch.empty(rows + 1, dtype=torch.int32, device=dev)
    kv_idx = torch.empty(rows * nKb, dtype=torch.int32, device=dev)
    ws_sel = torch.empty(max(1, losa.binding._select_workspace_bytes(wl.B, wl.H, wl.nQb, nKb)),
                         dtype=torch.uint8, device=dev)
    ws_attn = torch.empty(max(losa.losa_workspace_bytes(2, prob), losa.losa_workspace_bytes(3, prob)),
                          dtype=torch.uint8, device=dev)
    ws_fused = torch.empty(losa.losa_workspace_bytes(4, prob), dtype=torch.uint8, device=dev)
    mass_fused = torch.empty_like(mass)
    o_sparse = torch.empty_like(draws[0][0])
    o_dense = torch.empty_like(draws[0][0])

    def ev():
        return torch.cuda.Event(enable_timing=True)

    def step(record=None):
        marks = [ev()]
        marks[0].record()
        losa.losa_block_mass(q0d, k0d, wl.R, wl.C, ws=ws_mass, mass=mass)
        marks.append(ev()); marks[-1].record()
        losa.losa_select(mass, tau, ws=ws_sel, out=(offsets, kv_idx))
        marks.append(ev()); marks[-1].record()
        for (q, k, v) in draws:
            losa.losa_sparse_attn(q, k, v, offsets, kv_idx, wl.R, wl.C, out=o_sparse, ws=ws_attn)
            marks.append(ev()); marks[-1].record()
        q, k, v = draws[0]
        losa.losa_attn(q, k, v, wl.R, wl.C, out=o_dense, ws=ws_attn)
        marks.append(ev()); marks[-1].record()
        losa.losa_attn_mass(q, k, v, wl.R, wl.C, out=o_dense, mass=mass_fused, ws=ws_fused)
        marks.append(ev()); marks[-1].record()
        if record is not None:
            record.append(marks)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    losa.check_async("warm-up")
    off_h = offsets.cpu().numpy()
    idx_h = kv_idx[: int(off_h[-1])].cpu().numpy()
    flops_sparse = retained_flops(wl, off_h, idx_h)
    coverage = float(off_h[-1]) / float(rows * nKb)

    records = []
    barrier()
    with ClockSampler(local_rank) as clocks:
        t_start, t_end = ev(), ev()
        t_start.record()
        for _ in range(args.steps):
            step(records)
        t_end.record()
        barrier()
    losa.check_async("timed region")
    total_ms = t_start.elapsed_time(t_end)

    mass_ms, sel_ms, sparse_ms, dense_ms, fused_ms = [], [], [], [], []
    for marks in records:
        mass_ms.append(marks[0].elapsed_time(marks[1]))
        sel_ms.append(marks[1].elapsed_time(marks[2]))
        for i in range(args.draws):
            sparse_ms.append(marks[2 + i].elapsed_time(marks[3 + i]))
        dense_ms.append(marks[2 + args.draws].elapsed_time(marks[3 + args.draws]))
        fused_ms.append(marks[3 + args.draws].elapsed_time(marks[4 + args.draws]))
    sparse_total_ms = sum(sparse_ms)

    total_ms_max, sparse_total_ms_max = max_over_ranks([total_ms, sparse_total_ms], dist, dev)
    n_sparse_calls = args.steps * args.draws
    if shard_heads:
        # strong scaling: the job is ONE layer; its flops are the sum of the ranks' shares
        flops_job = sum_over_ranks(flops_sparse, dist, dev)
        value = flops_job * n_sparse_calls / (sparse_total_ms_max * 1e-3) / 1e12
    else:
        value = aggregate_tflops(flops_sparse, n_sparse_calls, sparse_total_ms_max, world)

    # ---- Recall (Eq. 2) of the frozen pattern: at the construction step and on every reuse draw
    # (outside the timed region: it needs the block masses of every draw)
    def recall_of(qd_, kd_):
        m = losa.losa_block_mass(qd_, kd_, wl.R, wl.C, ws=ws_mass, mass=mass_fused)
        ret, tot = losa.losa_row_recall(m, offsets, kv_idx)
        return float(ret.sum() / tot.sum()), float((ret / tot).min())

    recall0 = recall_of(q0d, k0d)
    recall_draws = [recall_of(d[0], d[1]) for d in draws]
    losa.check_async("recall")
    gpu_mass_h = mass.cpu().numpy().reshape(rows, nKb)

    # ---- several layers in one launch against the same layers one call each (optional)
    batched = None
    if args.batched_layers > 1:
        L = args.batched_layers
        layers = [draws[i % len(draws)] + (offsets, kv_idx) for i in range(L)]
        outs = [torch.empty_like(draws[0][0]) for _ in range(L)]
        ws_b = torch.empty(losa.losa_workspace_bytes_batched(2, prob, L), dtype=torch.uint8, device=dev)

        def timed(fn, reps=20):
            for _ in range(3):
                fn()
            a, b = ev(), ev()
            a.record()
            for _ in range(reps):
                fn()
            b.record()
            torch.cuda.synchronize()
            return a.elapsed_time(b) / reps

        def singles():
            for (q, k, v, o_, i_), o in zip(layers, outs):
                losa.losa_sparse_attn(q, k, v, o_, i_, wl.R, wl.C, out=o, ws=ws_attn)

        ms_single = timed(singles)
        ms_batched = timed(lambda: losa.losa_sparse_attn_batched(layers, wl.R, wl.C, outs=outs, ws=ws_b))
        losa.check_async("batched")
        batched = {"layers": L, "ms_single_calls": ms_single, "ms_one_launch": ms_batched,
                   "speedup": ms_single / ms_batched}

    # ---- end to end through the public API with host buffers (pinned), copies inside the timing
    e2e = None
    if not args.no_e2e:
        pin = [tuple(t.pin_memory() for t in d) for d in host_draws]
        q0p, k0p = q0.pin_memory(), k0.pin_memory()
        o_host = torch.empty(o_sparse.shape, dtype=o_sparse.dtype).pin_memory()
        # two sets of device buffers: while the kernels work on one, a copy stream fills the other
        # and drains the previous output (what a caller that feeds the library from host memory does)
        bufs = [tuple(torch.empty_like(draws[0][0]) for _ in range(4)) for _ in range(2)]  # q, k, v, o
        h2d_stream = torch.cuda.Stream(device=dev)   # inputs: host -> device
        d2h_stream = torch.cuda.Stream(device=dev)   # outputs: device -> host (the link is full duplex)
        main_stream = torch.cuda.current_stream()

        def e2e_step():
            ready = [torch.cuda.Event() for _ in range(2)]      # inputs of a buffer set have landed
            computed = [torch.cuda.Event() for _ in range(2)]   # kernels are done with a buffer set
            drained = [None, None]                              # its output has been copied back
            qd, kd = bufs[0][0], bufs[0][1]
            qd.copy_(q0p, non_blocking=True)
            kd.copy_(k0p, non_blocking=True)
            losa.losa_block_mass(qd, kd, wl.R, wl.C, ws=ws_mass, mass=mass)
            losa.losa_select(mass, tau, ws=ws_sel, out=(offsets, kv_idx))
            computed[0].record(main_stream)
            for t, (q, k, v) in enumerate(pin):
                s_ = t & 1
                qd, kd, vd, od = bufs[s_]
                with torch.cuda.stream(h2d_stream):
                    if t >= 2 or t == 0:
                        h2d_stream.wait_event(computed[s_])     # the last kernel that read this set is done
                    qd.copy_(q, non_blocking=True)
                    kd.copy_(k, non_blocking=True)
                    vd.copy_(v, non_blocking=True)
                    ready[s_].record(h2d_stream)
                main_stream.wait_event(ready[s_])
                if drained[s_] is not None:
                    main_stream.wait_event(drained[s_])         # this set's previous output is on the host
                losa.losa_sparse_attn(qd, kd, vd, offsets, kv_idx, wl.R, wl.C, out=od, ws=ws_attn)
                computed[s_] = torch.cuda.Event()
                computed[s_].record(main_stream)
                with torch.cuda.stream(d2h_stream):
                    d2h_stream.wait_event(computed[s_])
                    o_host.copy_(od, non_blocking=True)
                    drained[s_] = torch.cuda.Event()
                    drained[s_].record(d2h_stream)
            main_stream.wait_stream(d2h_stream)                 # the step ends with its last output on the host
            main_stream.wait_stream(h2d_stream)

        e2e_step()
        barrier()
        a, b = ev(), ev()
        n_e2e = max(1, min(args.steps, 2))
        a.record()
        for _ in range(n_e2e):
            e2e_step()
        b.record()
        barrier()
        (e2e_ms,) = max_over_ranks([a.elapsed_time(b)], dist, dev)
        nbytes = q0.numel() * 2
        e2e = {
            "value": (sum_over_ranks(flops_sparse, dist, dev) * args.draws * n_e2e / (e2e_ms * 1e-3) / 1e12
                      if shard_heads else aggregate_tflops(flops_sparse, args.draws * n_e2e, e2e_ms, world)),
            "unit": UNIT,
            "h2d_bytes_per_step": (2 + 3 * args.draws) * nbytes,
            "d2h_bytes_per_step": args.draws * nbytes,
            "ms_per_step": e2e_ms / n_e2e,
            "steps": n_e2e,
            "note": "mass+select+draws x sparse attention; every call's q/k/v copied from pinned "
                    "host memory and every output copied back inside the timed region; copies run on "
                    "two more streams (one per direction) into double-buffered device tensors and "
                    "overlap the kernels",
        }
        losa.check_async("e2e")

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    sparse_avg_ms = sparse_total_ms / n_sparse_calls
    achieved = flops_sparse / (sparse_avg_ms * 1e-3) / 1e12
    burst = float(peaks["bf16_tflops"])
    sustained = float(peaks.get("bf16_tflops_sustained", burst))
    dense_flops = wl.dense_flop()
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": total_ms_max / args.steps, "higher_is_better": True,
        "scaling": "strong" if shard_heads else "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {
            "workload": wl.name, "B": wl.B, "H": full_heads, "N": wl.N, "D": wl.D, "R": wl.R, "C": wl.C,
            "tau": tau, "draws": args.draws, "coverage": coverage, "nnz": int(off_h[-1]),
            "step": "block_mass + select + draws x sparse_attn + 1 dense attn + 1 fused attn_mass",
            "l2": "inputs larger than L2: each sparse call reads a different 300 MB draw",
            "pe_base": wl.pe_base, "pe_scale": wl.pe_scale,
            "multi_gpu": ("heads of one layer split across the ranks (rank 0 reports its own share "
                          f"of {wl.H} heads below)" if shard_heads else
                          "every rank its own layer" if world > 1 else "one GPU"),
        },
        "ms_per_layer": {
            "sparse_attn": sparse_avg_ms, "sparse_attn_min": min(sparse_ms),
            "dense_attn": statistics.mean(dense_ms), "block_mass": statistics.mean(mass_ms),
            "select": statistics.mean(sel_ms),
            "attn_mass_fused": statistics.mean(fused_ms),
        },
        "sparse_vs_dense_speedup": statistics.mean(dense_ms) / sparse_avg_ms,
        "dense_tflops": dense_flops / (statistics.mean(dense_ms) * 1e-3) / 1e12,
        "block_mass_tflops": 0.5 * dense_flops / (statistics.mean(mass_ms) * 1e-3) / 1e12,
        "select_gbs": (4.0 * rows * nKb + 4.0 * (int(off_h[-1]) + rows + 1)) / (statistics.mean(sel_ms) * 1e-3) / 1e9,
        "recall": {
            "construction_step": recall0[0], "construction_step_min_row": recall0[1],
            "reuse_draws": [r[0] for r in recall_draws], "reuse_draws_min_row": [r[1] for r in recall_draws],
            "note": "Eq. 2 on the GPU's own block masses of each draw, frozen pattern from step 0",
        },
        "roofline": {
            "kernel": "losa_attn_kernel<sparse>", "bound": "tensor", "achieved": achieved,
            "peak": burst, "unit": "TFLOP/s", "frac": achieved / burst,
            "peak_source": f"{peaks['_source']} bf16_tflops (cuBLAS burst)",
            "frac_of_sustained": achieved / sustained,
            "frac_of_nominal": achieved / NOMINAL_BF16_TFLOPS,
            "flops_per_launch": flops_sparse,
            "traffic": NCU_DRAM_BYTES_PER_LAUNCH.get(wl.name),
            "traffic_unit": "bytes per launch (DRAM read + write)",
            "traffic_source": NCU_TRAFFIC_SOURCE if wl.name in NCU_DRAM_BYTES_PER_LAUNCH else None,
            "algorithmic_bytes_per_launch": 4 * q0.numel() * 2,
        },
        "clocks": clocks.summary(),
        "gpu_launches": args.steps * launches_per_step(wl, args.draws),
    }
    if batched is not None:
        line["batched"] = batched
    if e2e is not None:
        line["e2e"] = e2e
    if not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(wl, *host_draws[0], off_h, idx_h, args.cpu_seconds,
                                            gpu_mass=gpu_mass_h, tau=tau)
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

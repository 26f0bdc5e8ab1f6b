#!/usr/bin/env python
"""Benchmark of the Hotline hot path on B200: samples/s through fragment + embedding-bag forward/backward
(+ cold gather/scatter), one process per GPU, synthetic inputs.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

A "step" is one mini-batch through the whole path: hl_fragment, hl_gather_cold (side stream), hl_embbag_fwd and
hl_embbag_bwd_sgd for the popular and then the non-popular micro-batch, hl_scatter_cold.  Rank 0 prints ONE JSON
line.  `--impl reference` times the CPU oracle on the host cores instead (rank 0 only).
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

import gen  # noqa: E402

METRIC = "samples/sec through fragment+embbag fwd/bwd"
UNIT = "samples/s"
L2_BYTES = 126 << 20
FALLBACK_HBM_GBS = 6650.0          # earlier measurement on this machine, used only if MEASURED_PEAKS.json is absent
SINGLE_ALLOCATION_LIMIT = 64 << 30  # a larger host table is held as one allocation per table


def log(*a):
    print(*a, file=sys.stderr, flush=True)


# ----------------------------------------------------------------------------------------------------------
# workload
# ----------------------------------------------------------------------------------------------------------
def mem_available_bytes() -> int:
    try:
        for line in open("/proc/meminfo"):
            if line.startswith("MemAvailable"):
                return int(line.split()[1]) * 1024
    except OSError:
        pass
    return 0


def pick_workload(requested: str, world: int):
    """(config name, row scale).  The metric is quoted on the DLRM-large-like configuration; every rank keeps its
    own host table, so with several ranks (or little host RAM) the table is shrunk, or DLRM-small-like is used."""
    if requested != "auto":
        return requested, 1.0
    need = gen.make_geometry(gen.CONFIGS["dlrm_large"]).total_rows * 64 * 4
    avail = mem_available_bytes()
    if avail and need * world <= 0.7 * avail:
        return "dlrm_large", 1.0
    return "dlrm_small", 1.0


def max_nnz_of(spec, geom) -> int:
    bags = geom.num_tables * spec.batch * geom.bags_per_sample
    return bags if spec.pooling[0] == "one" else bags * int(spec.pooling[2])


def fill_table(table, dim: int, seed: int, device, chunk_rows: int = 1 << 21, integer: bool = False,
               row0: int = 0) -> None:
    """table[i, :] = gen.table_values(row0 + i) for every row, computed on the device in chunks and copied down."""
    import torch
    n = table.shape[0]
    for r0 in range(0, n, chunk_rows):
        r1 = min(n, r0 + chunk_rows)
        table[r0:r1].copy_(gen.table_values_torch(row0 + r0, r1 - r0, dim, seed, device, integer=integer))
    if str(device) != "cpu":
        torch.cuda.synchronize()


class Workload:
    """Everything both arms need: geometry, the host table, profiling and timed batches (host copies)."""

    def __init__(self, name: str, scale: float, n_batches: int, profile_batches, device, threads: int,
                 with_table: bool = True):
        self.spec = gen.CONFIGS[name]
        self.geom = gen.make_geometry(self.spec, scale)
        self.name, self.scale = name, scale
        g, s = self.geom, self.spec
        self.T, self.D, self.S, self.B, self.N = g.num_tables, g.dim, g.bags_per_sample, s.batch, g.total_rows
        self.n_bags = self.T * self.B * self.S
        self.max_nnz = max_nnz_of(s, g)
        self.P = s.profile_batches if profile_batches is None else profile_batches
        self.hot_cap = max(1, min(self.N, self._policy_rows()))
        self.staging_cap = max(1, min(self.N, self.max_nnz))
        self.table = None
        if with_table:       # the CUDA arm's host table: memory the device can address, filled from the device
            import paper_2204_05436_b200 as hl
            t0 = time.time()
            if self.N * self.D * 4 > SINGLE_ALLOCATION_LIMIT:
                # above what one large-page allocation takes: one allocation per table (hl_set_host_tables)
                self.table = [hl.host_table_tensor(r, self.D) for r in g.table_rows]
                for t, ten in enumerate(self.table):
                    fill_table(ten, self.D, s.seed, device, row0=int(g.base[t]))
            else:
                self.table = hl.host_table_tensor(self.N, self.D)
                fill_table(self.table, self.D, s.seed, device)
            log(f"[bench] host table {self.N} x {self.D} fp32 = {self.N * self.D * 4 / 2**30:.1f} GiB "
                f"({len(self.table) if isinstance(self.table, list) else 1} allocation(s)) filled in "
                f"{time.time() - t0:.1f}s")
        t0 = time.time()
        self.profile = [gen.make_batch(s, g, i, threads) for i in range(self.P)]
        self.batches = [gen.make_batch(s, g, self.P + i, threads) for i in range(n_batches)]
        log(f"[bench] drew {self.P} profiling + {n_batches} timed batches in {time.time() - t0:.1f}s")

    def _policy_rows(self) -> int:
        p = self.spec.hot_policy
        if p[0] == "budget":
            return int(p[1]) // (4 * self.D)
        if p[0] == "fraction":
            return self.N * int(p[1]) // int(p[2])
        return int(p[1])

    def policy_args(self):
        import paper_2204_05436_b200 as hl
        p = self.spec.hot_policy
        if p[0] == "budget":
            return hl.HL_HOT_BUDGET_BYTES, int(p[1]), 1
        if p[0] == "fraction":
            return hl.HL_HOT_FRACTION_ROWS, int(p[1]), int(p[2])
        return hl.HL_HOT_TOPK_ROWS, int(p[1]), 1

    def free(self):
        if self.table is None:
            return
        import paper_2204_05436_b200 as hl
        ptrs = [t.data_ptr() for t in (self.table if isinstance(self.table, list) else [self.table])]
        self.table = None
        for ptr in ptrs:
            hl.hl_host_free(ptr)


# ----------------------------------------------------------------------------------------------------------
# clocks
# ----------------------------------------------------------------------------------------------------------
class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML (read-only) every few milliseconds."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, gpu_index: int, period_s: float = 0.004):
        self.period = period_s
        self.samples, self.reasons = [], set()
        self.stop_flag = threading.Event()
        self.thread = None
        self.handle = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            vis = os.environ.get("CUDA_VISIBLE_DEVICES")
            idx = int(vis.split(",")[gpu_index]) if vis and vis.split(",")[gpu_index].isdigit() else gpu_index
            self.handle = pynvml.nvmlDeviceGetHandleByIndex(idx)
            self.sm_max = float(pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM))
        except Exception as e:   # noqa: BLE001
            self.err = repr(e)

    def _run(self):
        nv = self.nv
        while not self.stop_flag.is_set():
            try:
                self.samples.append(float(nv.nvmlDeviceGetClockInfo(self.handle, nv.NVML_CLOCK_SM)))
                mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.handle))
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:   # noqa: BLE001
                pass
            time.sleep(self.period)

    def start(self):
        if self.handle is not None:
            self.thread = threading.Thread(target=self._run, daemon=True)
            self.thread.start()

    def stop(self) -> dict:
        if self.thread is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0, "reasons": ["NVML unavailable"]}
        self.stop_flag.set()
        self.thread.join(timeout=2)
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None, "sm_max_mhz": self.sm_max,
                "samples": len(self.samples), "reasons": sorted(self.reasons)}


# ----------------------------------------------------------------------------------------------------------
# CPU oracle legs (cpu_baseline of the CUDA arm, and the whole `--impl reference` arm)
# ----------------------------------------------------------------------------------------------------------
def take_samples(batch: gen.Batch, T: int, B: int, S: int, n: int, first: int = 0) -> gen.Batch:
    """Inputs first .. first+n of a table-major CSR mini-batch, as a mini-batch of n inputs."""
    if n >= B and first == 0:
        return batch
    off = batch.offsets.astype(np.int64)
    idx_parts, sizes = [], []
    for t in range(T):
        lo_bag, hi_bag = (t * B + first) * S, (t * B + first + n) * S
        idx_parts.append(batch.indices[off[lo_bag]:off[hi_bag]])
        sizes.append(np.diff(off[lo_bag:hi_bag + 1]))
    new_off = np.concatenate([[0], np.cumsum(np.concatenate(sizes))]).astype(np.int32)
    dense = None if batch.dense is None else batch.dense[first:first + n]
    return gen.Batch(np.concatenate(idx_parts).astype(np.int32), new_off, dense, n)


class OracleRunner:
    """Runs the CPU oracle, as it stands, on the workload: learning phase once, then one step per call.
    ``table``: fp32 [N, D] array-like holding (at least) the rows the steps will stage."""

    def __init__(self, wl, table, profile=None):
        from oracle import hotline_oracle as orc
        self.orc, self.wl = orc, wl
        t0 = time.time()
        profile = wl.profile if profile is None else profile
        cnt = orc.access_counts([(b.indices, b.offsets) for b in profile], wl.B, wl.geom.table_rows, wl.S)
        k = min(wl.hot_cap, orc.hot_capacity(wl.spec.hot_policy, wl.N, wl.D))
        self.hot = orc.select_hot(cnt, k)
        del cnt
        self.remap = orc.build_remap(self.hot, wl.N)
        self.table = table
        self.cache = None
        self.rng = np.random.default_rng(1234)
        log(f"[bench] oracle learning phase: {len(self.hot)} hot rows in {time.time() - t0:.1f}s")

    def load_cache(self, hot_values=None):
        wl = self.wl
        self.cache = np.zeros((wl.hot_cap + wl.staging_cap, wl.D), dtype=np.float32)
        self.cache[: len(self.hot)] = (self.orc.load_hot_cache(self.table, self.hot) if hot_values is None
                                       else hot_values)

    def sizes(self, batch: gen.Batch) -> dict:
        """What the index-only part of the path finds for this mini-batch (for the cross-check with the device)."""
        wl, orc = self.wl, self.orc
        _, n_pop, O, X, _ = orc.fragment(batch.indices, batch.offsets, batch.batch, wl.geom.table_rows, self.remap, wl.S)
        C, _ = orc.gather_cold(X.ids, self.remap, wl.hot_cap)
        return dict(n_pop=n_pop, n_non=batch.batch - n_pop, L_pop=len(O.ids), L_non=len(X.ids), n_cold=len(C), C=C)

    def step(self, batch: gen.Batch, cache=None):
        """(seconds, sizes) of one mini-batch through the oracle (fragment, gather, fwd/bwd of O and X, scatter)."""
        wl, orc = self.wl, self.orc
        n_bags = wl.T * batch.batch * wl.S
        grad = self.rng.standard_normal((n_bags, wl.D), dtype=np.float32)
        # the split of the gradient rows between O and X is input marshalling, outside the timed part
        _, n_pop, _, _, _ = orc.fragment(batch.indices, batch.offsets, batch.batch, wl.geom.table_rows, self.remap,
                                         wl.S)
        bags_pop = wl.T * n_pop * wl.S
        t0 = time.perf_counter()
        out = orc.hotline_step(self.table, self.cache if cache is None else cache, wl.hot_cap, self.remap,
                               batch.indices, batch.offsets, batch.batch, wl.geom.table_rows, wl.S, grad[:bags_pop],
                               grad[bags_pop:], wl.spec.lr)
        dt = time.perf_counter() - t0
        _, n_pop, O, X, C, _, _ = out
        return dt, dict(n_pop=n_pop, n_non=batch.batch - n_pop, L_pop=len(O.ids), L_non=len(X.ids), n_cold=len(C))

    def step_all_cores(self, batch: gen.Batch, cores: int) -> float:
        """Seconds for one mini-batch when its inputs are dealt out to ``cores`` threads, each running the oracle's
        step on its share (numpy releases the interpreter lock inside its array operations).  The threads share the
        tables and the staging area without coordination, so this leg times the work and its results are not used."""
        from concurrent.futures import ThreadPoolExecutor
        wl, orc = self.wl, self.orc
        per = -(-batch.batch // cores)
        shares = [take_samples(batch, wl.T, wl.B, wl.S, min(per, batch.batch - f), f)
                  for f in range(0, batch.batch, per)]
        rngs = [np.random.default_rng(99 + i) for i in range(len(shares))]

        def work(i):
            sh = shares[i]
            n_bags = wl.T * sh.batch * wl.S
            grad = rngs[i].standard_normal((n_bags, wl.D), dtype=np.float32)
            _, n_pop, _, _, _ = orc.fragment(sh.indices, sh.offsets, sh.batch, wl.geom.table_rows, self.remap, wl.S)
            bags_pop = wl.T * n_pop * wl.S
            orc.hotline_step(self.table, self.cache, wl.hot_cap, self.remap, sh.indices, sh.offsets, sh.batch,
                             wl.geom.table_rows, wl.S, grad[:bags_pop], grad[bags_pop:], wl.spec.lr)

        t0 = time.perf_counter()
        with ThreadPoolExecutor(max_workers=cores) as pool:
            list(pool.map(work, range(len(shares))))
        return time.perf_counter() - t0


def host_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:   # pragma: no cover
        return os.cpu_count() or 1


def sparse_oracle_table(wl, rows_needed: np.ndarray, tmpdir: str):
    """fp32 [N, D] table for the oracle that costs memory only for the rows in ``rows_needed``: a sparse file mapped
    into memory, those rows filled from the procedural initialiser (the same values the real table holds)."""
    table = np.memmap(os.path.join(tmpdir, "oracle_table.f32"), dtype=np.float32, mode="w+", shape=(wl.N, wl.D))
    rows_needed = np.asarray(rows_needed, dtype=np.int64)
    for i in range(0, len(rows_needed), 1 << 18):
        chunk = rows_needed[i:i + (1 << 18)]
        table[chunk] = gen.table_values(chunk, wl.D, wl.spec.seed)
    return table


def run_reference(args, rank: int, world: int) -> None:
    """The CPU oracle on the host cores, on the CUDA arm's workload.  Needs neither the library nor a GPU: the table
    is a sparse file holding the rows the sampled mini-batches stage."""
    if rank != 0:
        return
    import tempfile
    name, scale = pick_workload(args.workload, 1)
    if args.row_scale is not None:
        scale = args.row_scale
    wl = Workload(name, scale, n_batches=min(8, args.steps + args.warmup), profile_batches=args.profile_batches,
                  device=None, threads=args.threads, with_table=False)
    with tempfile.TemporaryDirectory() as tmp:
        runner = OracleRunner(wl, table=None)
        # size the per-step sample so that the whole run ends within a few minutes
        n_try = min(wl.B, 2048)
        probe = take_samples(wl.batches[0], wl.T, wl.B, wl.S, n_try)
        need = [runner.sizes(probe)["C"]]
        runner.table = sparse_oracle_table(wl, need[0], tmp)
        hot_values = gen.table_values(runner.hot, wl.D, wl.spec.seed)
        runner.load_cache(hot_values)
        t_probe, _ = runner.step(probe)
        budget = 150.0 / max(1, args.steps + args.warmup)
        n = int(min(wl.B, max(256, probe.batch * budget / max(t_probe, 1e-6))))
        n = 1 << (n.bit_length() - 1) if n < wl.B else wl.B
        sample = [take_samples(b, wl.T, wl.B, wl.S, n) for b in wl.batches]
        rows = np.unique(np.concatenate([runner.sizes(b)["C"] for b in sample]))
        del runner.table
        runner.table = sparse_oracle_table(wl, rows, tmp)
        runner.load_cache(hot_values)
        for i in range(args.warmup):
            runner.step(sample[i % len(sample)])
        times = [runner.step(sample[(args.warmup + i) % len(sample)])[0] for i in range(args.steps)]
        total = sum(times)
        value = n * args.steps / total
        sample_txt = f"first {n} of {wl.B} inputs of each mini-batch, {args.steps} mini-batches"
        line = {
            "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(wl, extra={"sample_inputs_per_step": n}),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample_txt},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0,
        }
        print(json.dumps(line), flush=True)
        del runner.table


def workload_config(wl, extra=None) -> dict:
    """The keys of `config` that name the workload; both arms print the same ones."""
    c = {"workload": wl.name, "row_scale": wl.scale, "batch": wl.B, "tables": wl.T, "dim": wl.D,
         "bags_per_sample": wl.S, "total_rows": wl.N, "table_gib": round(wl.N * wl.D * 4 / 2 ** 30, 2),
         "hot_cap_rows": wl.hot_cap, "profile_batches": wl.P}
    if extra:
        c.update(extra)
    return c


# ----------------------------------------------------------------------------------------------------------
# ranks: independent replicas, one per GPU; the only exchange is the barrier and the max of the timings
# ----------------------------------------------------------------------------------------------------------
def max_over_ranks(values, world: int, device="cpu"):
    """Element-wise maximum of ``values`` (floats) over all ranks of the default process group."""
    if world <= 1:
        return [float(v) for v in values]
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(v) for v in values], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.tolist()]


def whole_job_value(batch: int, steps: int, world: int, ms_total_max: float) -> float:
    """Samples per second of the whole job: every rank processed batch*steps inputs in the slowest rank's time."""
    return batch * world * steps / (ms_total_max * 1e-3)


def spawn_ranks(argv, n: int) -> int:
    """`python bench.py --gpus N` outside a launcher: starts the N ranks itself (one process per GPU)."""
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr",
           "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)
    return subprocess.run(cmd).returncode


# ----------------------------------------------------------------------------------------------------------
# CUDA arm
# ----------------------------------------------------------------------------------------------------------
# DRAM bytes (read + written) per bag of the forward kernel at dim 64, from a profiler capture of the hot-only
# micro case (`--micro fwd`: 425,984 one-lookup bags, 164.4 MB of DRAM traffic); a launch of the benchmark is
# scaled from it by its number of bags, since the traffic grows in proportion to the bags.
PROFILED_FWD_DRAM_BYTES_PER_BAG = {64: 164.4e6 / 425984}


def fwd_bytes(L, bags, D):
    """Algorithmic bytes of one forward launch: per lookup a row and its slot, per bag a pooled row and an offset."""
    return L * (4 * D + 4) + bags * (4 * D + 4)


def chunks_bytes(L, distinct, D):
    """Algorithmic bytes of the backward's sum kernel: per lookup a gradient row and its (slot, bag) pair, per
    distinct row one read-modify-write."""
    return L * (4 * D + 8) + distinct * 2 * 4 * D


def summarise_spans(spans):
    """Mean duration (us) per span kind, and per (kind, position among the same kind inside a mini-batch)."""
    by_kind, seq = {}, {}
    for sp in spans:
        key = (sp["mini_batch"], sp["name"])
        k = seq.get(key, 0)
        seq[key] = k + 1
        by_kind.setdefault((sp["name"], k), []).append((sp["end_ms"] - sp["begin_ms"]) * 1e3)
    return {f"{name}#{k}" if any(kk > 0 for (nn, kk) in by_kind if nn == name) else name:
            round(statistics.mean(v), 2) for (name, k), v in sorted(by_kind.items())}


def timeline_text(spans, mini_batches):
    """The spans of the given mini-batches as text, one line per span, ordered by begin time."""
    rows = sorted((sp for sp in spans if sp["mini_batch"] in mini_batches), key=lambda sp: sp["begin_ms"])
    if not rows:
        return ""
    t0 = rows[0]["begin_ms"]
    names = {0: "main", 1: "frag", 2: "sort", 3: "cold", 4: "read", 5: "wb"}
    out = ["   begin_us      end_us   dur_us  stream  mini-batch  what"]
    for sp in rows:
        out.append(f"{(sp['begin_ms'] - t0) * 1e3:10.1f}  {(sp['end_ms'] - t0) * 1e3:10.1f}  "
                   f"{(sp['end_ms'] - sp['begin_ms']) * 1e3:7.1f}  {names.get(sp['stream'], sp['stream']):>6}  "
                   f"{sp['mini_batch']:10d}  {sp['name']}")
    return "\n".join(out)


def run_cuda(args, rank: int, local_rank: int, world: int) -> None:
    import torch
    import torch.distributed as dist
    import paper_2204_05436_b200 as hl

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    device = torch.device(f"cuda:{local_rank}")
    torch.cuda.set_device(device)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)

    name, scale = pick_workload(args.workload, world)
    if args.row_scale is not None:
        scale = args.row_scale       # a labelled variant: every table shrunk by this factor
    n_batches = 16                   # distinct pre-generated mini-batches the timed steps rotate over
    wl = Workload(name, scale, n_batches, args.profile_batches, device, args.threads)
    T, D, S, B = wl.T, wl.D, wl.S, wl.B
    pipelined = not args.no_pipeline
    native = pipelined and not (args.python_pipeline or args.serial_link)
    eq5 = args.order == "eq5"
    if eq5 and not native:
        raise SystemExit("--order eq5 is a mode of the library's own scheduler")
    if native:
        h = hl.NativePipelinedHotline(wl.geom.table_rows, D, S, B, wl.max_nnz, wl.hot_cap, wl.staging_cap, wl.table,
                                      n_dense=wl.spec.n_dense, device=str(device), lookahead=args.lookahead,
                                      order=args.order, main_priority=args.main_priority,
                                      index_priority=args.index_priority, link_priority=args.link_priority,
                                      mover_ctas=args.mover_ctas, scatter_ctas=args.scatter_ctas,
                                      write_back=args.write_back)
    elif pipelined:
        h = hl.PipelinedHotline(wl.geom.table_rows, D, S, B, wl.max_nnz, wl.hot_cap, wl.staging_cap, wl.table,
                                n_dense=wl.spec.n_dense, device=str(device), overlap_link=not args.serial_link,
                                lookahead=args.lookahead, main_priority=args.main_priority,
                                side_priority=args.index_priority)
    else:
        h = hl.Hotline(wl.geom.table_rows, D, S, B, wl.max_nnz, wl.hot_cap, wl.staging_cap, wl.table,
                       n_dense=wl.spec.n_dense, device=str(device), main_priority=args.main_priority,
                       side_priority=args.index_priority)
        if args.mover_ctas or args.scatter_ctas:
            hl.hl_set_mover_ctas(h.ctx, args.mover_ctas, args.scatter_ctas)
    lr = wl.spec.lr
    sms = torch.cuda.get_device_properties(device).multi_processor_count
    if args.fwd_ctas or args.bwd_ctas:
        hl.hl_set_kernel_width(h.ctx, args.fwd_ctas, args.bwd_ctas)

    with torch.cuda.stream(h.main):
        # ---- learning phase (setup, timed separately) ----
        t0 = time.time()
        for i, b in enumerate(wl.profile):
            h.profile(torch.from_numpy(b.indices).to(device), torch.from_numpy(b.offsets).to(device), B, reset=(i == 0))
        pol, p_num, p_den = wl.policy_args()
        h.profile(None, None, finalize=True, policy=pol, p_num=p_num, p_den=p_den)
        h.build_remap(load_rows=True)
        h.status()
        n_hot = int(h.n_hot.item())
        log(f"[bench] learning phase on the device: {n_hot} hot rows of {wl.hot_cap} slots in {time.time() - t0:.1f}s")

        # ---- resident inputs ----
        pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()   # noqa: E731
        h_idx = [pin(b.indices) for b in wl.batches]
        h_off = [pin(b.offsets) for b in wl.batches]
        h_dense = [pin(b.dense) if b.dense is not None else None for b in wl.batches]
        d_idx = [x.to(device) for x in h_idx]
        d_off = [x.to(device) for x in h_off]
        d_dense = [x.to(device) if x is not None else None for x in h_dense]
        gen_t = torch.Generator(device=device)
        gen_t.manual_seed(wl.spec.seed + 1000 + rank)
        d_grad = torch.randn((wl.n_bags, D), generator=gen_t, device=device, dtype=torch.float32)
        h_grad = d_grad.cpu().pin_memory()
        torch.cuda.synchronize()

        cursor = [0]   # mini-batches issued so far; mini-batch i uses input buffers i % n_batches
        inputs = {"idx": d_idx, "off": d_off, "dense": d_dense}

        def batch_args(k):
            return (inputs["idx"][k], inputs["off"][k], B, inputs["dense"][k])

        def one_step(timers=None):
            """Issues the next mini-batch; returns (its buffer index k, the object holding its outputs)."""
            i = cursor[0]
            cursor[0] += 1
            k = i % n_batches
            if pipelined:
                if h.idle:
                    h.start(*batch_args(k), more=[batch_args((i + a) % n_batches) for a in range(1, h.lookahead)],
                            inputs_ready="resident")
                s = h.step(d_grad, None if eq5 else d_grad, lr, next_batch=batch_args((i + h.lookahead) % n_batches),
                           timers=timers, inputs_ready="resident")   # the timed region's inputs are in HBM already
                return k, h.sets[s]
            h.step(inputs["idx"][k], inputs["off"][k], B, d_grad, d_grad, lr, dense=inputs["dense"][k], timers=timers)
            return k, h

        def finish():
            """Everything issued so far is complete, write-backs included."""
            if pipelined:
                h.drain()
            torch.cuda.synchronize()

        def restart():
            """Empties the pipeline and realigns the rotation, so that the next step is mini-batch 0 of the rotation."""
            while pipelined and not h.idle:
                h.step(d_grad, None if eq5 else d_grad, lr, next_batch=None, inputs_ready="resident")
            finish()
            cursor[0] = 0

        def sizing_pass():
            """Per-batch sizes (they depend only on the indices and the hot set): one untimed pass."""
            out = [None] * n_batches
            restart()
            for _ in range(n_batches):
                k, o = one_step()
                finish()
                h.status()
                c = o.counts.cpu().tolist()
                pop_ids = o.pop_ids[:c[2]] if hasattr(o, "pop_ids") else None
                non_ids = o.non_ids[:c[3]] if hasattr(o, "non_ids") else None
                out[k] = dict(n_pop=c[0], n_non=c[1], L_pop=c[2], L_non=c[3], n_cold=int(o.n_cold.item()),
                              U_pop=int(torch.unique(pop_ids).numel()) if pop_ids is not None else 0,
                              U_non=int(torch.unique(non_ids[non_ids >= 0]).numel()) if non_ids is not None else 0)
            return out

        BW_MASK = 0
        if native:
            BW_MASK = (1 << 6) | (1 << 8) | (1 << (hl.HL_SPAN_KERNEL + hl.HL_TIMER_BWD_REDUCE))

        def timed_block(n_steps, mask=0, barrier=False):
            """n_steps steps between two events on the main stream, a synchronisation on both sides.
            Returns (ms, host enqueue us per step, spans, index of the first mini-batch)."""
            torch.cuda.synchronize()
            if barrier and world > 1:
                dist.barrier()
            if mask:
                h.trace_begin(16 * n_steps + 64, mask)
            ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            first = (cursor[0], h.j_done if pipelined else 0)     # position in the rotation, the schedule's own count
            timers = {"only": ("fwd_pop", "fwd_non")} if not native else None
            ev0.record(h.main)
            host_t0 = time.perf_counter()
            for _ in range(n_steps):
                one_step(timers)
            host_us = (time.perf_counter() - host_t0) / n_steps * 1e6
            if pipelined:
                h.wait_outputs()     # the last write-backs belong to the timed work
            ev1.record(h.main)
            finish()
            spans = h.trace_end() if mask else []
            if barrier and world > 1:
                dist.barrier()
            return ev0.elapsed_time(ev1), host_us, spans, first, timers

        sizes = sizing_pass()

        # ---- timed region: device-resident inputs ----
        for i in range(args.warmup):
            one_step()
        launches0 = hl.hl_launch_count()
        log(f"[bench] library kernel launches before the timed region: {launches0}")
        clocks = ClockSampler(local_rank)
        clocks.start()
        # The timed block carries no events between its kernels (in the library's scheduler; the Python schedulers
        # time their two forward calls as before): recording them costs about a tenth of the throughput.  The
        # in-step time of every bandwidth-bound kernel comes from the next block, the same steps again with an event
        # pair around those kernels.
        ms_total, host_enqueue_us, bw_spans, first_timed, fwd_timers = timed_block(args.steps, 0, barrier=True)
        launches = hl.hl_launch_count() - launches0
        h.status()
        ms_traced = None
        if native:
            ms_traced, _, bw_spans, first_timed, _ = timed_block(args.steps, BW_MASK)
            ms_traced /= args.steps
        # ---- the same block repeated, for a spread (each with a synchronisation on both sides, no events) ----
        block_ms = [ms_total / args.steps]
        for _ in range(args.blocks):
            ms, _, _, _, _ = timed_block(args.steps)
            block_ms.append(ms / args.steps)
        clock_info = clocks.stop()
        h.status()

        # ---- every call of the schedule, in place: a traced pass over n_batches steps (outside the timed region) ----
        all_spans, call_timers = [], {}
        if native:
            _, _, all_spans, first_traced, _ = timed_block(n_batches, hl.HL_SPAN_ALL)
        else:
            for _ in range(n_batches):
                one_step(call_timers)
            finish()

        # ---- kernels alone: nothing else on the chip, L2 flushed by a 256 MB write before every launch ----
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=device)
        restart()
        k_last, o_last = one_step()
        while pipelined and not h.idle:      # the last mini-batch stepped is the one whose buffers are used below
            o_last = h.sets[h.step(d_grad, None if eq5 else d_grad, lr, next_batch=None, inputs_ready="resident")]
            k_last += 1
        finish()
        sz_last = sizes[k_last % n_batches]
        stream = h.main.cuda_stream

        def alone(fn, reps=7):
            us = []
            for _ in range(reps):
                flush.zero_()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(h.main)
                fn()
                b.record(h.main)
                h.main.synchronize()
                us.append(a.elapsed_time(b) * 1e3)
            return statistics.median(us)

        alone_us = {
            "fwd_non": alone(lambda: hl.hl_embbag_fwd(h.ctx, h.cache, o_last.non, o_last.counts_non, o_last.pooled_non,
                                                      stream)),
            "fwd_pop": alone(lambda: hl.hl_embbag_fwd(h.ctx, h.cache, o_last.pop, o_last.counts, o_last.pooled_pop,
                                                      stream)),
        }
        # the movers alone at full width (two CTAs per multiprocessor) on that mini-batch's cold rows: reading them
        # again and writing them back again changes nothing (the pipeline is empty, the rows were written back)
        w_last = ((h.j_done - 1) % 2) * h.window_rows if pipelined else 0
        rows_last = h.window_rows if pipelined else h.staging_cap
        hl.hl_set_mover_ctas(h.ctx, 2 * sms, 2 * sms)
        alone_us["move_read"] = alone(lambda: hl.hl_stage_cold(h.ctx, h.host_table, h.cache, w_last, rows_last,
                                                               o_last.cold_rows, o_last.n_cold, None, stream))
        alone_us["move_write"] = alone(lambda: hl.hl_scatter_cold_at(h.ctx, h.cache, w_last, rows_last,
                                                                     o_last.cold_rows, o_last.n_cold, h.host_table,
                                                                     stream))
        hl.hl_set_mover_ctas(h.ctx, args.mover_ctas, args.scatter_ctas)
        h.status()
        del flush
        link = {}
        buf_h = torch.empty(256 << 20, dtype=torch.uint8).pin_memory()
        buf_d = torch.empty(256 << 20, dtype=torch.uint8, device=device)
        for nm, (dst, src) in {"h2d": (buf_d, buf_h), "d2h": (buf_h, buf_d)}.items():
            best = 0.0
            for _ in range(5):
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                dst.copy_(src, non_blocking=True)
                b.record()
                torch.cuda.synchronize()
                best = max(best, buf_h.numel() / (a.elapsed_time(b) * 1e-3) / 1e9)
            link[nm] = best
        del buf_h, buf_d

        # ---- hot-only run: the same mini-batches with every lookup redirected into the profiled popular set, so
        # that every input is popular and nothing crosses the host link (the hot embedding-bag by itself) ----
        hot_only = None
        if not args.no_hot_only:
            hot_rows_np = h.hot_rows[:n_hot].cpu().numpy()
            hb = [gen.restrict_to_rows(b, wl.geom, hot_rows_np) for b in wl.batches]
            if all(x is not None for x in hb):
                restart()
                inputs["idx"] = [torch.from_numpy(x.indices).to(device) for x in hb]
                torch.cuda.synchronize()
                hot_sizes = sizing_pass()
                for _ in range(max(3, args.warmup)):
                    one_step()
                ms_hot, _, hot_spans, first_hot, hot_timers = timed_block(args.steps, 0)
                if native:        # the kernels' in-step times from a repetition with events, as for the main run
                    _, _, hot_spans, first_hot, _ = timed_block(args.steps, BW_MASK)
                hot_only = dict(ms=ms_hot, spans=hot_spans, first=first_hot, sizes=hot_sizes, timers=hot_timers)
                restart()
                inputs["idx"] = d_idx
                torch.cuda.synchronize()
                h.status()

        # ---- end to end: host buffers in, results out, copies inside the timed region ----
        e2e = None
        if not args.no_e2e:
            restart()
            out_pop = torch.empty((wl.n_bags, D), dtype=torch.float32).pin_memory()
            out_non = torch.empty((wl.n_bags, D), dtype=torch.float32).pin_memory()
            out_counts = torch.empty(4, dtype=torch.int32).pin_memory()
            out_perm = torch.empty(B, dtype=torch.int32).pin_memory()
            h2d = d2h = 0

            def e2e_step(i):
                # the inputs copied here are those of the mini-batch whose ahead-work this step issues (pipelined)
                # or of this step's own mini-batch (sequential); the gradients are this step's
                nonlocal h2d, d2h
                k = ((cursor[0] + h.lookahead) if pipelined else cursor[0]) % n_batches
                d_idx[k].copy_(h_idx[k], non_blocking=True)
                d_off[k].copy_(h_off[k], non_blocking=True)
                h2d_now = h_idx[k].numel() * 4 + h_off[k].numel() * 4 + h_grad.numel() * 4
                if d_dense[k] is not None:
                    d_dense[k].copy_(h_dense[k], non_blocking=True)
                    h2d_now += h_dense[k].numel() * 4
                d_grad.copy_(h_grad, non_blocking=True)
                _k, o = one_step()
                out_counts.copy_(o.counts, non_blocking=True)
                out_perm.copy_(o.perm[:B], non_blocking=True)
                h.main.synchronize()
                bags_pop, bags_non = T * int(out_counts[0]) * S, T * int(out_counts[1]) * S
                out_pop[:bags_pop].copy_(o.pooled_pop[:bags_pop], non_blocking=True)
                out_non[:bags_non].copy_(o.pooled_non[:bags_non], non_blocking=True)
                h.main.synchronize()
                h2d, d2h = h2d_now, 16 + B * 4 + (bags_pop + bags_non) * D * 4

            if pipelined:
                # The copies are pipelined like the work: while mini-batch j executes, the gradients of j+1 and the
                # indices of j+lookahead come in on one copy stream and the outputs of j-1 go out on another (the
                # link carries both directions at once).  Every step's inputs and outputs cross the link inside the
                # timed region; gradients and host output buffers are double-buffered.
                s_in, s_out, s_cnt = (torch.cuda.Stream(device=device) for _ in range(3))
                d_grads = [d_grad, torch.empty_like(d_grad)]
                outs = [(out_pop, out_non, out_counts, out_perm),
                        (torch.empty_like(out_pop).pin_memory(), torch.empty_like(out_non).pin_memory(),
                         torch.empty_like(out_counts).pin_memory(), torch.empty_like(out_perm).pin_memory())]
                ev_in = [torch.cuda.Event() for _ in range(2)]
                ev_grad_free = [torch.cuda.Event() for _ in range(2)]
                ev_out = [torch.cuda.Event() for _ in range(2)]
                ev_done, ev_cnt = torch.cuda.Event(), torch.cuda.Event()
                for e in ev_grad_free + ev_out:
                    e.record(h.main)
                L = h.lookahead

                def e2e_pipe_step(i):
                    nonlocal h2d, d2h
                    j = cursor[0]
                    cursor[0] += 1
                    kin, g = (j + L) % n_batches, i % 2
                    with torch.cuda.stream(s_in):
                        s_in.wait_event(ev_grad_free[g])          # the backward of two steps ago has read this buffer
                        d_idx[kin].copy_(h_idx[kin], non_blocking=True)
                        d_off[kin].copy_(h_off[kin], non_blocking=True)
                        h2d_now = h_idx[kin].numel() * 4 + h_off[kin].numel() * 4 + h_grad.numel() * 4
                        if d_dense[kin] is not None:
                            d_dense[kin].copy_(h_dense[kin], non_blocking=True)
                            h2d_now += h_dense[kin].numel() * 4
                        d_grads[g].copy_(h_grad, non_blocking=True)
                        ev_in[g].record(s_in)
                    h.main.wait_event(ev_in[g])               # this step's gradients
                    if h.idle:
                        h.start(*batch_args(j % n_batches),
                                more=[batch_args((j + a) % n_batches) for a in range(1, L)])
                    st = h.sets[h.step(d_grads[g], None if eq5 else d_grads[g], lr, next_batch=batch_args(kin),
                                       inputs_ready=ev_in[g])]
                    ev_grad_free[g].record(h.main)
                    ev_done.record(h.main)
                    o_pop, o_non, o_counts, o_perm = outs[g]
                    ev_out[g].synchronize()                       # the outputs of two steps ago have left this buffer
                    with torch.cuda.stream(s_cnt):                # sizes of this mini-batch: known since its fragment
                        h.wait_counts(s_cnt)
                        o_counts.copy_(st.counts, non_blocking=True)
                        ev_cnt.record(s_cnt)
                    ev_cnt.synchronize()
                    bags_pop, bags_non = T * int(o_counts[0]) * S, T * int(o_counts[1]) * S
                    assert int(o_counts[0]) + int(o_counts[1]) == B, "fragment counts do not add up to the mini-batch"
                    with torch.cuda.stream(s_out):
                        s_out.wait_event(ev_done)
                        o_perm.copy_(st.perm[:B], non_blocking=True)
                        o_pop[:bags_pop].copy_(st.pooled_pop[:bags_pop], non_blocking=True)
                        o_non[:bags_non].copy_(st.pooled_non[:bags_non], non_blocking=True)
                        ev_out[g].record(s_out)
                    h2d, d2h = h2d_now, 16 + B * 4 + (bags_pop + bags_non) * D * 4

                step_fn = e2e_pipe_step
            else:
                step_fn = e2e_step
            for i in range(max(3, min(args.warmup, 5))):
                step_fn(i)
            torch.cuda.synchronize()
            if world > 1:
                dist.barrier()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            finish()
            torch.cuda.synchronize()
            e0.record(h.main)
            for i in range(args.steps):
                step_fn(args.warmup + i)
            if pipelined:
                h.wait_outputs()
                h.main.wait_stream(s_out)
            e1.record(h.main)
            finish()
            torch.cuda.synchronize()
            e2e_ms = e0.elapsed_time(e1)
            e2e = {"ms_total": e2e_ms, "h2d": h2d, "d2h": d2h}
        h.status()

    # ---- reduce over ranks (max time) ----
    red = max_over_ranks([ms_total, e2e["ms_total"] if e2e else 0.0], world, device)
    ms_total = red[0]
    if e2e:
        e2e["ms_total"] = red[1]

    if rank == 0:
        ms_per_step = ms_total / args.steps
        value = whole_job_value(B, args.steps, world, ms_total)
        peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
        if os.path.exists(peaks_path):
            peak, peak_src = float(json.load(open(peaks_path))["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
        else:
            peak, peak_src = FALLBACK_HBM_GBS, "fallback"

        def kernel_table(spans, timers, first, n_steps, sz):
            """In-step time and fraction of the HBM peak of each bandwidth-bound kernel of a step: both forward
            launches and the backward's two sum kernels, from the events recorded inside the timed block."""
            used = [sz[(first[0] + i) % n_batches] for i in range(n_steps)]
            mean = lambda key: sum(u[key] for u in used) / len(used)   # noqa: E731
            dur = {}
            if spans:
                seq = {}
                for sp in spans:
                    nm = sp["name"]
                    if nm == "k_bwd_chunks":
                        k = seq.get(sp["mini_batch"], 0)
                        seq[sp["mini_batch"]] = k + 1
                        nm = "bwd_chunks_all" if eq5 else ("bwd_chunks_pop" if k == 0 else "bwd_chunks_non")
                    dur.setdefault(nm, []).append((sp["end_ms"] - sp["begin_ms"]) * 1e3)
            elif timers:
                for nm in ("fwd_pop", "fwd_non"):
                    dur[nm] = [a.elapsed_time(b) * 1e3 for a, b in timers.get(nm, [])]
            bags_pop, bags_non = T * mean("n_pop") * S, T * mean("n_non") * S
            algo = {"fwd_pop": fwd_bytes(mean("L_pop"), bags_pop, D), "fwd_non": fwd_bytes(mean("L_non"), bags_non, D),
                    "bwd_chunks_pop": chunks_bytes(mean("L_pop"), mean("U_pop"), D),
                    "bwd_chunks_non": chunks_bytes(mean("L_non"), mean("U_non"), D),
                    "bwd_chunks_all": chunks_bytes(mean("L_pop") + mean("L_non"), mean("U_pop") + mean("U_non"), D)}
            table = {}
            for nm, v in dur.items():
                if not v or nm not in algo:
                    continue
                us = statistics.mean(v)
                gbs = algo[nm] / (us * 1e-6) / 1e9 if us > 0 else 0.0
                table[nm] = {"algorithmic_bytes_per_launch": algo[nm], "us_per_launch": us, "launches": len(v),
                             "achieved": gbs, "frac": gbs / peak}
            return table, mean, bags_pop, bags_non

        kt, mean, bags_pop, bags_non = kernel_table(bw_spans, fwd_timers, first_timed, args.steps, sizes)
        # The roofline line is the hot embedding-bag forward: both forward launches of a step taken together (the
        # popular micro-batch's rows in the hot cache, and the non-popular one's over hot cache + staged rows, all
        # in HBM), algorithmic bytes over the in-step time of the two launches.
        f_us = sum(kt[k]["us_per_launch"] for k in ("fwd_pop", "fwd_non") if k in kt)
        f_bytes = sum(kt[k]["algorithmic_bytes_per_launch"] for k in ("fwd_pop", "fwd_non") if k in kt)
        achieved = f_bytes / (f_us * 1e-6) / 1e9 if f_us > 0 else 0.0
        per_bag = PROFILED_FWD_DRAM_BYTES_PER_BAG.get(D)

        def alone_entry(nm, L, bags):
            us = alone_us[nm]
            gbs = fwd_bytes(L, bags, D) / (us * 1e-6) / 1e9
            return {"us_per_launch": us, "achieved": gbs, "frac": gbs / peak}

        roofline = {"kernel": "k_embbag_fwd, both launches of a step (popular + non-popular micro-batch)",
                    "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                    "peak_source": peak_src, "traffic": per_bag * (bags_pop + bags_non) if per_bag else None,
                    "traffic_source": "profiler capture of the hot-only micro case, scaled by bags",
                    "algorithmic_bytes_per_launch": f_bytes, "us_per_launch": f_us,
                    "note": "us_per_launch = sum of the two forward launches of a step, timed by CUDA events on the "
                            "main stream in a repetition of the timed block (the same steps again, right after it, with "
                            "an event pair around each bandwidth-bound kernel), where they share the chip with the other "
                            "streams; the timed block itself runs without those events",
                    "ms_per_step_of_that_block": ms_traced,
                    "kernels_in_step": kt,
                    "alone": {"note": "the same launches over one mini-batch with nothing else on the chip, L2 flushed",
                              "fwd_non": alone_entry("fwd_non", sz_last["L_non"], T * sz_last["n_non"] * S),
                              "fwd_pop": alone_entry("fwd_pop", sz_last["L_pop"], T * sz_last["n_pop"] * S)}}
        # host link: the movers' kernels in the traced pass (in step) and alone at full width
        move = {"k_move_read": [], "k_move_write": []}
        for sp in all_spans:
            if sp["name"] in move:      # which mini-batch of the rotation the span's mini-batch is
                k = (first_traced[0] + sp["mini_batch"] - first_traced[1]) % n_batches
                move[sp["name"]].append(((sp["end_ms"] - sp["begin_ms"]) * 1e3, sizes[k]["n_cold"]))

        def link_entry(v, peak_gbs):
            if not v:
                return None
            us = statistics.mean(t for t, _ in v)
            gbs = statistics.mean(n * D * 4 / (t * 1e-6) / 1e9 for t, n in v if t > 0)
            return {"kernel_us": us, "gbs": gbs, "frac_of_memcpy": gbs / peak_gbs}

        bytes_last = sz_last["n_cold"] * D * 4
        host_link = {
            "memcpy_h2d_gbs": link["h2d"], "memcpy_d2h_gbs": link["d2h"],
            "cold_rows_per_step": mean("n_cold"), "bytes_per_step": mean("n_cold") * D * 4,
            "in_step": {"read": link_entry(move["k_move_read"], link["h2d"]),
                        "write_back": link_entry(move["k_move_write"], link["d2h"]),
                        "note": "the movers' kernels inside the schedule, next to the other streams' kernels"},
            "alone": {"rows": sz_last["n_cold"],
                      "read": {"kernel_us": alone_us["move_read"], "gbs": bytes_last / alone_us["move_read"] / 1e3,
                               "frac_of_memcpy": bytes_last / alone_us["move_read"] / 1e3 / link["h2d"]},
                      "write_back": {"kernel_us": alone_us["move_write"],
                                     "gbs": bytes_last / alone_us["move_write"] / 1e3,
                                     "frac_of_memcpy": bytes_last / alone_us["move_write"] / 1e3 / link["d2h"]},
                      "note": "one mini-batch's cold rows, two mover CTAs per multiprocessor, nothing else running"}}
        breakdown = summarise_spans(all_spans) if all_spans else \
            {k: round(1e3 * sum(a.elapsed_time(b) for a, b in v) / max(1, len(v)), 2) for k, v in call_timers.items()}
        if all_spans and args.timeline:
            os.makedirs(os.path.dirname(os.path.abspath(args.timeline)), exist_ok=True)
            mbs = sorted({sp["mini_batch"] for sp in all_spans})
            with open(args.timeline, "w") as f:
                f.write(timeline_text(all_spans, set(mbs[len(mbs) // 2: len(mbs) // 2 + 3])) + "\n")
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": workload_config(wl, extra={
                "hot_rows": n_hot, "popular_fraction": round(mean("n_pop") / B, 4),
                "cold_rows_per_step": round(mean("n_cold"), 1),
                "l2": "no explicit flush: a step reads and writes more than the 126 MB L2 "
                      f"({(2 * wl.n_bags * D * 4 + f_bytes) / 2**20:.0f} MB of pooled vectors, gradients and rows)"
                      if 2 * wl.n_bags * D * 4 > L2_BYTES else
                      "per-step working set is smaller than L2 on this workload; batches rotate over 16 buffers",
                "schedule": ("software-pipelined across mini-batches ("
                             + ("hl_pipe_*, issued by the library" if native else "PipelinedHotline, issued from Python")
                             + (", host reads after write-backs)" if args.serial_link else
                                ", host reads overlap write-backs, shared rows forwarded)")
                             + ("; order of Eq. 5: both forwards, then one update per row and mini-batch"
                                if eq5 else "")
                             if pipelined else "one mini-batch after the other (Hotline.step)"),
                "stream_priorities": {"main": args.main_priority, "index": args.index_priority,
                                      "link": args.link_priority},
                "mover_ctas": {"read": args.mover_ctas or "default", "write": args.scatter_ctas or "default"},
                "write_back": args.write_back,
                "replicas": "independent replica per GPU, no collective"}),
            "clocks": clock_info, "gpu_launches": int(launches), "host_enqueue_us_per_step": host_enqueue_us,
            "launches_per_step": launches / args.steps,
            "blocks": {"note": f"the timed block of {args.steps} steps and {args.blocks} repetitions of it, each "
                               "synchronised on both sides; ms per step",
                       "n": len(block_ms), "median": statistics.median(block_ms), "min": min(block_ms),
                       "max": max(block_ms)},
            "breakdown_us": breakdown, "roofline": roofline, "host_link": host_link,
        }
        if hot_only:
            hk, hmean, hb_pop, _ = kernel_table(hot_only["spans"], hot_only["timers"], hot_only["first"], args.steps,
                                                hot_only["sizes"])
            line["hot_only"] = {
                "note": "the same schedule on the same mini-batches with every lookup redirected into the profiled "
                        "popular set: every input is popular, nothing crosses the host link",
                "ms_per_step": hot_only["ms"] / args.steps, "value": B * args.steps / (hot_only["ms"] * 1e-3),
                "popular_fraction": hmean("n_pop") / B, "cold_rows_per_step": hmean("n_cold"), "kernels_in_step": hk}
        if e2e:
            line["e2e"] = {"value": B * world * args.steps / (e2e["ms_total"] * 1e-3), "unit": UNIT,
                           "h2d_bytes_per_step": e2e["h2d"], "d2h_bytes_per_step": e2e["d2h"],
                           "ms_per_step": e2e["ms_total"] / args.steps}
        if world == 1 and not args.no_cpu_baseline:
            h.close()
            if isinstance(wl.table, list):
                # per-table allocations: the oracle gets a sparse table holding the rows its mini-batches stage
                import tempfile
                tmp = tempfile.TemporaryDirectory()
                runner = OracleRunner(wl, None)
                need = np.unique(np.concatenate([runner.sizes(b)["C"] for b in wl.batches[:2]]))
                runner.table = sparse_oracle_table(wl, need, tmp.name)
                runner.load_cache(gen.table_values(runner.hot, D, wl.spec.seed))
                oracle_batches = wl.batches[:2]
            else:
                runner = OracleRunner(wl, wl.table.numpy())
                runner.load_cache()
                oracle_batches = wl.batches
            times, checked = [], 0
            for i, b in enumerate(oracle_batches):
                dt, sz = runner.step(b)
                times.append(dt)
                # the oracle is the checker of what was timed: the sizes the device found for this mini-batch
                for key in ("n_pop", "n_non", "L_pop", "L_non", "n_cold"):
                    if sz[key] != sizes[i][key]:
                        raise SystemExit(f"[bench] mini-batch {i}: device {key} = {sizes[i][key]}, oracle {sz[key]}")
                checked += 1
                if sum(times) > 15.0:
                    break
            line["cpu_baseline"] = {"value": B * len(times) / sum(times), "unit": UNIT, "cores": 1, "kind": "oracle",
                                    "sample": f"{len(times)} whole mini-batches of {B} inputs ({sum(times):.1f} s)",
                                    "cross_check": f"n_pop, n_non, L_pop, L_non, n_cold of {checked} timed mini-batches "
                                                   "equal the device's"}
            cores = min(host_cores(), 32)
            if cores > 1:
                t_all = [runner.step_all_cores(wl.batches[i % len(wl.batches)], cores) for i in range(4)]
                line["cpu_baseline"]["all_cores"] = {
                    "value": B * len(t_all) / sum(t_all), "unit": UNIT, "cores": cores, "kind": "oracle",
                    "sample": f"{len(t_all)} whole mini-batches, inputs dealt out to {cores} threads that each run "
                              f"the oracle's step on their share ({sum(t_all):.1f} s)"}
        print(json.dumps(line), flush=True)
    h.close()
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    wl.free()


# ----------------------------------------------------------------------------------------------------------
# single-call micro runs (small cases: one library call in isolation, sized for a profiler capture)
# ----------------------------------------------------------------------------------------------------------
def run_micro_gather(args) -> None:
    """`--micro gather`: the row-move kernel alone, host table -> HBM and back, 65,536 rows of 256 bytes of a 16 GiB
    host table: consecutive rows, random rows within the first 4 GiB, random rows over the whole table; each
    pattern is gathered three times (the later repetitions find their address translations resident) and then
    written back three times (hl_flush_hot: the same mover in the other direction)."""
    import torch
    import paper_2204_05436_b200 as hl
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    N, D, K = 1 << 26, 64, 1 << 16
    table = hl.host_table_tensor(N, D)
    h = hl.Hotline([N], D, 1, 64, 64, K, 16, table)
    rng = np.random.default_rng(0)
    cases = {"consecutive": np.arange(K), "random_4GiB": np.sort(rng.choice(1 << 24, K, replace=False)),
             "random_16GiB": np.sort(rng.choice(N, K, replace=False))}
    buf_h = torch.empty(256 << 20, dtype=torch.uint8).pin_memory()
    buf_d = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    best = 0.0
    for _ in range(5):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        buf_d.copy_(buf_h, non_blocking=True)
        b.record()
        torch.cuda.synchronize()
        best = max(best, buf_h.numel() / (a.elapsed_time(b) * 1e-3) / 1e9)
    best_d2h = 0.0
    for _ in range(5):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        buf_h.copy_(buf_d, non_blocking=True)
        b.record()
        torch.cuda.synchronize()
        best_d2h = max(best_d2h, buf_h.numel() / (a.elapsed_time(b) * 1e-3) / 1e9)
    res = {"micro": "gather", "rows": K, "row_bytes": 4 * D, "table_gib": N * D * 4 / 2 ** 30, "memcpy_h2d_gbs": best,
           "memcpy_d2h_gbs": best_d2h}

    def timed(load):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(h.main)
        h.build_remap(load_rows=load)
        b.record(h.main)
        torch.cuda.synchronize()
        return a.elapsed_time(b)

    with torch.cuda.stream(h.main):
        for name, rows in cases.items():
            h.set_hot_rows(torch.from_numpy(rows).to(dev))
            torch.cuda.synchronize()
            base = min(timed(False) for _ in range(3))          # remap kernels without the row load
            runs = [timed(True) - base for _ in range(3)]
            res[name] = {"first_gbs": K * D * 4 / runs[0] / 1e6, "best_gbs": K * D * 4 / min(runs) / 1e6,
                         "best_frac_of_memcpy": K * D * 4 / min(runs) / 1e6 / best}
            wb = []
            for _ in range(3):
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(h.main)
                h.flush_hot()
                b.record(h.main)
                torch.cuda.synchronize()
                wb.append(a.elapsed_time(b))
            res[name]["write_back"] = {"first_gbs": K * D * 4 / wb[0] / 1e6, "best_gbs": K * D * 4 / min(wb) / 1e6,
                                       "best_frac_of_memcpy": K * D * 4 / min(wb) / 1e6 / best_d2h}
    h.status()
    h.close()
    print(json.dumps(res), flush=True)
    hl.hl_host_free(table.data_ptr())


def run_micro_tracker(args) -> None:
    """`--micro tracker`: the approximate access logger (hl_tracker_*) next to the exact counters on the learning
    phase of the chosen workload (`--workload`, `--profile-batches` mini-batches): time per mini-batch of both, and
    how much of the exact popular set the logger finds -- for loggers of 1, 2 and 4 M blocks (16 ways; the paper's
    has 2 M blocks), each asked for 70 % of its blocks, against the exact top rows of the same number."""
    import torch
    import paper_2204_05436_b200 as hl
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    spec = gen.CONFIGS["dlrm_large" if args.workload in (None, "auto") else args.workload]
    geom = gen.make_geometry(spec, 1.0)
    T, D, S, B = geom.num_tables, spec.dim, geom.bags_per_sample, spec.batch
    N = int(sum(geom.table_rows))
    n_bags = T * B * S
    max_nnz = n_bags if spec.pooling[0] == "one" else n_bags * int(spec.pooling[2])
    P = args.profile_batches or 64
    block_counts = [1 << 20, 1 << 21, 1 << 22]
    hot_cap = int(0.7 * max(block_counts))
    g = hl.make_geometry(geom.table_rows, D, S)
    ws_bytes = hl.hl_workspace_bytes(g, B, max_nnz, hot_cap, 0)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
    ctx = hl.hl_create(g, B, max_nnz, hot_cap, 0, ws, ws_bytes)
    stream = torch.cuda.current_stream().cuda_stream
    base = torch.from_numpy(np.concatenate([[0], np.cumsum(geom.table_rows)]).astype(np.int64)).to(dev)
    batches = [gen.make_batch(spec, geom, i, args.threads) for i in range(P)]
    d_in = [(torch.from_numpy(b.indices).to(dev), torch.from_numpy(b.offsets).to(dev)) for b in batches]
    cnt = torch.zeros(N, dtype=torch.int64, device=dev)        # exact counts kept here too, to weigh the sets
    for idx, off in d_in:
        sizes = (off[1:] - off[:-1]).to(torch.int64)
        table = torch.arange(n_bags, device=dev) // (B * S)
        rows = base[torch.repeat_interleave(table, sizes)] + idx.to(torch.int64)
        cnt += torch.bincount(rows, minlength=N)
    total = float(cnt.sum().item())
    hot_rows = torch.zeros(hot_cap, dtype=torch.int32, device=dev)
    n_hot = torch.zeros(1, dtype=torch.int64, device=dev)

    def timed(fn):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) * 1e3

    def batch_of(i):
        return hl.make_batch(d_in[i][0], d_in[i][1], B, int(d_in[i][0].numel()))

    exact_us = [timed(lambda i=i: hl.hl_profile_hot(ctx, batch_of(i), int(i == 0), 0, 0, 0, 1, hot_rows, n_hot, stream))
                for i in range(P)]
    res = {"micro": "tracker", "workload": spec.name, "total_rows": N, "mini_batches": P, "lookups_per_mini_batch":
           int(d_in[0][0].numel()), "exact_counter_us_per_mini_batch": statistics.median(exact_us), "loggers": []}
    exact_sets = {}
    for blocks in block_counts:
        k = int(0.7 * blocks)
        hl.hl_profile_hot(ctx, None, 0, 1, hl.HL_HOT_TOPK_ROWS, k, 1, hot_rows, n_hot, stream)
        torch.cuda.synchronize()
        exact_sets[blocks] = hot_rows[:int(n_hot.item())].to(torch.int64).clone()
    for blocks in block_counts:
        ways, n_sets, k = 16, blocks // 16, int(0.7 * blocks)
        tags = torch.empty(blocks, dtype=torch.int32, device=dev)
        rrpv = torch.empty(blocks, dtype=torch.uint8, device=dev)
        hits = torch.zeros(1, dtype=torch.int64, device=dev)
        hl.hl_tracker_reset(ctx, tags, rrpv, n_sets, ways, hits, stream)
        us = [timed(lambda i=i: hl.hl_tracker_update(ctx, batch_of(i), tags, rrpv, n_sets, ways, hits, stream))
              for i in range(P)]
        hl.hl_tracker_export(ctx, tags, rrpv, n_sets, ways, stream)
        hl.hl_profile_hot(ctx, None, 0, 1, hl.HL_HOT_TOPK_ROWS, k, 1, hot_rows, n_hot, stream)
        torch.cuda.synchronize()
        tracked = hot_rows[:int(n_hot.item())].to(torch.int64)
        exact = exact_sets[blocks]
        mass_t, mass_e = float(cnt[tracked].sum().item()) / total, float(cnt[exact].sum().item()) / total
        common = int(torch.isin(tracked, exact).sum().item())
        res["loggers"].append({
            "blocks": blocks, "ways": ways, "asked_rows": k, "tracked_rows": int((tags >= 0).sum().item()),
            "selected_rows": int(tracked.numel()), "exact_rows": int(exact.numel()),
            "update_us_per_mini_batch": statistics.median(us), "update_us_max": max(us),
            "hit_rate": float(hits.item()) / (P * d_in[0][0].numel()),
            "captured_mass": mass_t, "exact_mass": mass_e, "mass_vs_exact": mass_t / mass_e if mass_e else None,
            "exact_rows_found": common / max(1, int(exact.numel()))})
    hl.hl_status(ctx)
    hl.hl_destroy(ctx)
    print(json.dumps(res), flush=True)


def run_micro_wide(args) -> None:
    """`--micro wide`: the index part of the path (learning phase, remap, fragment, cold-row search) through the
    wide-id calls (64-bit row ids, hashed counter, hashed remap) next to the same calls of the 32-bit path (dense
    counter, bitmap remap) on the same mini-batches of the chosen workload: time per call, CUDA events, and the
    outputs of the two paths compared (popular set, perm, counts, cold rows)."""
    import torch
    import paper_2204_05436_b200 as hl
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    n_timed = 8
    wl = Workload("dlrm_large" if args.workload in (None, "auto") else args.workload,
                  1.0 if args.row_scale is None else args.row_scale, n_timed, args.profile_batches or 64, dev,
                  args.threads, with_table=False)
    spec, geom = wl.spec, wl.geom
    T, D, S, B, N, P = wl.T, wl.D, wl.S, wl.B, wl.N, wl.P
    n_bags, max_nnz, hot_cap, staging = wl.n_bags, wl.max_nnz, wl.hot_cap, wl.staging_cap
    stream = torch.cuda.current_stream().cuda_stream
    i32, i64 = torch.int32, torch.int64
    batches = wl.profile + wl.batches
    d_in = [(torch.from_numpy(b.indices).to(dev), torch.from_numpy(b.offsets).to(dev)) for b in batches]
    policy, p_num, p_den = wl.policy_args()

    def batch_of(i):
        return hl.make_batch(d_in[i][0], d_in[i][1], B, int(d_in[i][0].numel()))

    def timed(fn):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) * 1e3

    z = lambda n, dt: torch.zeros(max(1, n), dtype=dt, device=dev)   # noqa: E731
    # ---- 32-bit path ----
    g = hl.make_geometry(geom.table_rows, D, S)
    ws_bytes = hl.hl_workspace_bytes(g, B, max_nnz, hot_cap, staging)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
    ctx = hl.hl_create(g, B, max_nnz, hot_cap, staging, ws, ws_bytes)
    hot32, n_hot32 = z(hot_cap, i32), z(1, i64)
    perm, counts = z(B, i32), z(4, i32)
    pop_off, pop_ids = z(n_bags + 1, i32), z(max_nnz, i32)
    non_off, non_ids = z(n_bags + 1, i32), z(max_nnz, i32)
    cold32, n_cold32 = z(staging, i32), z(1, i64)
    pop, non = hl.make_ubatch(pop_off, pop_ids, max_nnz), hl.make_ubatch(non_off, non_ids, max_nnz)
    t32 = {"profile": [timed(lambda i=i: hl.hl_profile_hot(ctx, batch_of(i), int(i == 0), 0, 0, 0, 1, hot32, n_hot32,
                                                           stream)) for i in range(P)]}
    t32["select"] = [timed(lambda: hl.hl_profile_hot(ctx, None, 0, 1, policy, p_num, p_den, hot32, n_hot32, stream))]
    t32["remap"] = [timed(lambda: hl.hl_build_remap(ctx, hot32, n_hot32, None, None, None, stream))]
    t32["fragment"], t32["index_cold"], out32 = [], [], []
    for rep in range(3):
        for i in range(P, P + n_timed):
            t32["fragment"].append(timed(lambda i=i: hl.hl_fragment(ctx, batch_of(i), None, 0, perm, counts, pop, non,
                                                                    None, stream)))
            t32["index_cold"].append(timed(lambda: hl.hl_index_cold(ctx, non, counts[1:], 0, staging, cold32, n_cold32,
                                                                    None, None, None, stream)))
            if rep == 0:
                nc = int(n_cold32.item())
                out32.append((perm.clone(), counts.clone(), cold32[:nc].to(i64).clone()))
    hl.hl_status(ctx)
    n_hot = int(n_hot32.item())
    hot32_rows = hot32[:n_hot].to(i64).clone()
    hl.hl_destroy(ctx)
    del ws
    # ---- wide path ----
    seen = int(torch.unique(torch.cat([_global_rows(torch, geom, B, S, idx, off, dev) for idx, off in d_in[:P]])).numel())
    counter_slots = 1 << max(16, (4 * seen - 1).bit_length())
    wws_bytes = hl.hl_wide_workspace_bytes(g, B, max_nnz, hot_cap, staging, counter_slots)
    wws = torch.empty(wws_bytes, dtype=torch.uint8, device=dev)
    w = hl.hl_wide_create(g, B, max_nnz, hot_cap, staging, counter_slots, wws, wws_bytes)
    hot64, n_hot64 = z(hot_cap, i64), z(1, i64)
    non_rows, non_slots = z(max_nnz, i64), z(max_nnz, i32)
    cold64, n_cold64 = z(staging, i64), z(1, i64)
    tw = {"profile": [timed(lambda i=i: hl.hl_wide_profile_hot(w, batch_of(i), i == 0, False, 0, 0, 1, 4 * D, hot64,
                                                               n_hot64, stream)) for i in range(P)]}
    tw["select"] = [timed(lambda: hl.hl_wide_profile_hot(w, None, False, True, policy, p_num, p_den, 4 * D, hot64,
                                                         n_hot64, stream))]
    tw["remap"] = [timed(lambda: hl.hl_wide_build_remap(w, hot64, n_hot64, stream))]
    tw["fragment"], tw["index_cold"] = [], []
    same = int(n_hot64.item()) == n_hot and bool(torch.equal(hot64[:n_hot], hot32_rows))
    for rep in range(3):
        for k, i in enumerate(range(P, P + n_timed)):
            tw["fragment"].append(timed(lambda i=i: hl.hl_wide_fragment(w, batch_of(i), perm, counts, pop, non_off,
                                                                        non_rows, max_nnz, stream)))
            tw["index_cold"].append(timed(lambda: hl.hl_wide_index_cold(w, non_off, non_rows, max_nnz, counts[1:],
                                                                        non_slots, cold64, n_cold64, stream)))
            if rep == 0:
                nc = int(n_cold64.item())
                same = same and bool(torch.equal(perm, out32[k][0]) and torch.equal(counts, out32[k][1])
                                     and torch.equal(cold64[:nc], out32[k][2]))
    hl.hl_wide_status(w)
    hl.hl_wide_destroy(w)
    med = lambda d: {k: round(statistics.median(v), 2) for k, v in d.items()}   # noqa: E731
    print(json.dumps({"micro": "wide", "workload": spec.name, "total_rows": N, "profile_mini_batches": P,
                      "lookups_per_mini_batch": int(d_in[0][0].numel()), "distinct_rows_seen": seen,
                      "counter_slots": counter_slots, "hot_rows": n_hot,
                      "cold_rows_per_mini_batch": round(statistics.mean(int(o[2].numel()) for o in out32), 1),
                      "us_per_call_32bit": med(t32), "us_per_call_wide": med(tw),
                      "same_results": same}), flush=True)


def _global_rows(torch, geom, B, S, idx, off, dev):
    """Global row id (table base + index) of every lookup of a table-major mini-batch."""
    base = torch.from_numpy(np.concatenate([[0], np.cumsum(geom.table_rows)]).astype(np.int64)).to(dev)
    n_bags = geom.num_tables * B * S
    sizes = (off[1:] - off[:-1]).to(torch.int64)
    table = torch.arange(n_bags, device=dev) // (B * S)
    return base[torch.repeat_interleave(table, sizes)] + idx.to(torch.int64)


def run_micro(args) -> None:
    """`--micro fwd|bwd`: one library call in isolation on an all-popular ("hot-only") micro-batch with the
    DLRM-large-like shape (26 tables x `--micro-batch` inputs, dim 64, one lookup per bag) over a 1 GiB cache.
    Slots are uniform over the cache (`--micro-dist uniform`: no reuse, every row comes from HBM) or Zipf(1.2)
    within each table's share of the cache (`zipf`: long runs of equal slots, as in the real workload)."""
    import torch
    import paper_2204_05436_b200 as hl
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    T, D, S, B = 26, args.micro_dim, 1, args.micro_batch
    H = (1 << 30) // (4 * D)
    n_bags = T * B
    rng = np.random.default_rng(5)
    if args.micro_dist == "uniform":
        ids = rng.integers(0, H, n_bags, dtype=np.int64)
    else:
        per = H // T
        ids = np.concatenate([t * per + gen.feistel_permute(gen.zipf_ranks(rng, 1.2, per, B) - 1, per, 17 + t)
                              for t in range(T)])
    geom = hl.make_geometry([H], D, 1)            # one "table" as large as the cache: slots are what matter here
    ws_bytes = hl.hl_workspace_bytes(geom, n_bags, n_bags, H, 0)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
    ctx = hl.hl_create(geom, n_bags, n_bags, H, 0, ws, ws_bytes)
    if args.fwd_ctas or args.bwd_ctas:
        hl.hl_set_kernel_width(ctx, args.fwd_ctas, args.bwd_ctas)
    cache = torch.rand((H, D), device=dev, dtype=torch.float32) - 0.5
    d_ids = torch.from_numpy(ids.astype(np.int32)).to(dev)
    d_off = torch.arange(n_bags + 1, dtype=torch.int32, device=dev)
    d_n = torch.tensor([n_bags], dtype=torch.int32, device=dev)
    out = torch.empty((n_bags, D), dtype=torch.float32, device=dev)
    grad = torch.randn((n_bags, D), dtype=torch.float32, device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    ub = hl.make_ubatch(d_off, d_ids, n_bags)
    stream = torch.cuda.current_stream().cuda_stream
    distinct = int(np.unique(ids).shape[0])
    if args.micro == "fwd":
        call = lambda: hl.hl_embbag_fwd(ctx, cache, ub, d_n, out, stream)   # noqa: E731
        nbytes = n_bags * (4 * D + 4) + n_bags * (4 * D + 4)
    else:
        call = lambda: hl.hl_embbag_bwd_sgd(ctx, cache, ub, d_n, grad, 1e-3, stream)   # noqa: E731
        nbytes = n_bags * (4 * D + 8) + distinct * 2 * 4 * D
    for _ in range(max(3, args.warmup)):
        call()
    times = []
    for _ in range(args.steps):
        flush.zero_()                      # write 256 MB: nothing of the previous call is left in the 126 MB L2
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        call()
        b.record()
        torch.cuda.synchronize()
        times.append(a.elapsed_time(b) * 1e3)
    hl.hl_status(ctx)
    us = statistics.median(times)
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    peak = float(json.load(open(peaks_path))["hbm_gbs"]) if os.path.exists(peaks_path) else FALLBACK_HBM_GBS
    print(json.dumps({"micro": args.micro, "dist": args.micro_dist, "bags": n_bags, "dim": D, "distinct_rows": distinct,
                      "us_median": us, "us_min": min(times), "algorithmic_bytes": nbytes,
                      "gbs": nbytes / us / 1e3, "frac_of_hbm_peak": nbytes / us / 1e3 / peak, "peak_gbs": peak,
                      "l2": "flushed between calls (256 MB write)"}), flush=True)
    hl.hl_destroy(ctx)


# ----------------------------------------------------------------------------------------------------------
# sensitivity sweeps on synthetic data (the paper's Section VII-F studies: popular / non-popular ratio, batch size)
# ----------------------------------------------------------------------------------------------------------
def run_sweep(args) -> None:
    """`--sweep`: (1) the hot-cache budget is cut from the configuration's value down to 1/64 of it, which moves
    the ratio of popular to non-popular inputs; (2) the mini-batch size is varied at the full budget.  Every point:
    10 warm-up and 60 timed mini-batches through the default pipeline, CUDA events.  Budget points also get the
    overlap efficiency of the host link (the paper's Section VII-F claim is that the gather stays hidden as the share
    of popular inputs falls): the same steps are timed with the whole table resident in HBM (the movers then move
    rows inside the device, which costs next to nothing), and the movers are timed alone on one mini-batch's rows;
    efficiency = 1 - (time with the host table - time with the resident table) / (read alone + write-back alone),
    i.e. the share of the transfers' own time that the schedule hides.  One JSON line."""
    import dataclasses
    import torch
    import paper_2204_05436_b200 as hl
    device = torch.device("cuda:0")
    torch.cuda.set_device(device)
    name, scale = pick_workload(args.workload, 1)
    if args.row_scale is not None:
        scale = args.row_scale
    wl = Workload(name, scale, 8, args.profile_batches, device, args.threads)
    T, D, S = wl.T, wl.D, wl.S
    sms = torch.cuda.get_device_properties(device).multi_processor_count
    points = []

    def measure(h, batches, B, n_bags, movers_alone=False):
        d_in = [(torch.from_numpy(b.indices).to(device), torch.from_numpy(b.offsets).to(device), B,
                 torch.from_numpy(b.dense).to(device) if b.dense is not None else None) for b in batches]
        d_grad = torch.randn((n_bags, D), device=device, dtype=torch.float32)
        torch.cuda.synchronize()
        n = len(d_in)
        it = [0]

        def step(last=False):
            i = it[0]
            it[0] += 1
            if h.idle:
                h.start(*d_in[i % n], more=[d_in[(i + a) % n] for a in range(1, h.lookahead)], inputs_ready="resident")
            return h.sets[h.step(d_grad, d_grad, wl.spec.lr, next_batch=None if last else d_in[(i + h.lookahead) % n],
                                 inputs_ready="resident")]

        pops, colds = [], []
        for _ in range(n):
            st = step()
            h.drain()
            pops.append(int(st.counts[0].item()))
            colds.append(int(st.n_cold.item()))
        for _ in range(10):
            step()
        h.drain()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(h.main)
        for _ in range(60):
            step()
        h.wait_outputs()
        e1.record(h.main)
        h.drain()
        h.status()
        out = dict(batch=B, popular_fraction=sum(pops) / (len(pops) * B), cold_rows_per_step=sum(colds) / len(colds),
                   ms_per_step=e0.elapsed_time(e1) / 60)
        while not h.idle:                 # empty the pipeline: the last mini-batch stepped is used below
            st = step(last=True)
        h.drain()
        if movers_alone:
            flush = torch.empty(256 << 20, dtype=torch.uint8, device=device)
            w = ((h.j_done - 1) % 2) * h.window_rows
            hl.hl_set_mover_ctas(h.ctx, 2 * sms, 2 * sms)

            def alone(fn):
                us = []
                for _ in range(5):
                    flush.zero_()
                    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    a.record(h.main)
                    fn()
                    b.record(h.main)
                    h.main.synchronize()
                    us.append(a.elapsed_time(b) * 1e3)
                return statistics.median(us)

            s_ = h.main.cuda_stream
            out["read_alone_us"] = alone(lambda: hl.hl_stage_cold(h.ctx, h.host_table, h.cache, w, h.window_rows,
                                                                  st.cold_rows, st.n_cold, None, s_))
            out["write_back_alone_us"] = alone(lambda: hl.hl_scatter_cold_at(h.ctx, h.cache, w, h.window_rows,
                                                                             st.cold_rows, st.n_cold, h.host_table, s_))
            out["alone_rows"] = int(st.n_cold.item())
            hl.hl_set_mover_ctas(h.ctx, 0, 0)
            h.status()
        return out

    def learn(h, k_rows):
        for i, b in enumerate(wl.profile):
            h.profile(torch.from_numpy(b.indices).to(device), torch.from_numpy(b.offsets).to(device), wl.B, reset=(i == 0))
        h.profile(None, None, finalize=True, policy=hl.HL_HOT_TOPK_ROWS, p_num=k_rows)
        h.build_remap(load_rows=True)
        h.status()
        return int(h.n_hot.item())

    def make(table, max_batch=None):
        mb = wl.B if max_batch is None else max_batch
        nnz = T * mb * S if wl.spec.pooling[0] == "one" else T * mb * S * int(wl.spec.pooling[2])
        return hl.NativePipelinedHotline(wl.geom.table_rows, D, S, mb, nnz, wl.hot_cap, min(wl.N, nnz), table,
                                         n_dense=wl.spec.n_dense, device=str(device))

    # (1) budget / ratio sweep, with the overlap efficiency of the link
    resident = None
    if not isinstance(wl.table, list):
        try:
            resident = torch.empty((wl.N, D), dtype=torch.float32, device=device)
            resident.copy_(wl.table, non_blocking=False)
        except RuntimeError:      # no room for a copy of the table in HBM: the sweep goes without the efficiency
            resident = None
    h = make(wl.table)
    h_res = make(resident) if resident is not None else None
    for div in (1, 2, 4, 16, 64):
        k = max(1, wl.hot_cap // div)
        with torch.cuda.stream(h.main):
            n_hot = learn(h, k)
            pt = measure(h, wl.batches, wl.B, wl.n_bags, movers_alone=True)
            h.flush_hot()            # the host table gets the popular rows back before the set changes
            h.status()
        pt.update(sweep="budget", budget_fraction=1.0 / div, hot_rows=n_hot, samples_per_s=wl.B / pt["ms_per_step"] * 1e3)
        if h_res is not None:
            with torch.cuda.stream(h_res.main):
                learn(h_res, k)
                res = measure(h_res, wl.batches, wl.B, wl.n_bags)
                h_res.flush_hot()
                h_res.status()
            scale_rows = pt["cold_rows_per_step"] / max(1, pt["alone_rows"])     # the alone run moved one mini-batch's rows
            t_link = (pt["read_alone_us"] + pt["write_back_alone_us"]) * 1e-3 * scale_rows
            pt["ms_per_step_table_resident"] = res["ms_per_step"]
            pt["link_alone_ms_per_step"] = t_link
            pt["overlap_efficiency"] = 1.0 - (pt["ms_per_step"] - res["ms_per_step"]) / t_link if t_link > 0 else None
        points.append(pt)
        log(f"[sweep] {pt}")
    h.close()
    if h_res is not None:
        h_res.close()
    del resident
    torch.cuda.empty_cache()
    # (2) batch-size sweep at the full budget
    for B in (2048, 4096, 8192, 32768):
        spec = dataclasses.replace(wl.spec, batch=B)
        batches = [gen.make_batch(spec, wl.geom, 100_000 + i, args.threads) for i in range(8)]
        h = make(wl.table, max(B, wl.B))
        with torch.cuda.stream(h.main):
            n_hot = learn(h, wl.hot_cap)
            pt = measure(h, batches, B, T * B * S)
            h.flush_hot()
            h.status()
        pt.update(sweep="batch", budget_fraction=1.0, hot_rows=n_hot, samples_per_s=B / pt["ms_per_step"] * 1e3)
        points.append(pt)
        log(f"[sweep] {pt}")
        h.close()
    print(json.dumps({"sweep": wl.name, "row_scale": wl.scale, "unit": "ms per mini-batch, samples/s",
                      "points": points}), flush=True)
    wl.free()


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--workload", default="auto", choices=["auto"] + sorted(gen.CONFIGS))
    ap.add_argument("--profile-batches", type=int, default=None)
    ap.add_argument("--row-scale", type=float, default=None,
                    help="shrink every table of the workload by this factor (a labelled variant, e.g. to reach the "
                         "share of popular inputs the paper reports)")
    ap.add_argument("--threads", type=int, default=min(16, os.cpu_count() or 1))
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-pipeline", action="store_true",
                    help="run one mini-batch after the other (Hotline.step) instead of the software pipeline "
                         "(PipelinedHotline), in which the next mini-batch's fragment, cold-row search and host reads "
                         "run under this one's execution")
    ap.add_argument("--serial-link", action="store_true",
                    help="pipeline variant in which the host read of the next mini-batch follows this one's write-back "
                         "instead of overlapping it (no forwarding of shared rows needed)")
    ap.add_argument("--lookahead", type=int, default=2,
                    help="mini-batches by which the index-only ahead-work of the pipelined schedule runs ahead")
    ap.add_argument("--python-pipeline", action="store_true",
                    help="issue the pipelined schedule from Python (PipelinedHotline) instead of the library's own "
                         "scheduler (hl_pipe_*); gives a time for every call in breakdown_us")
    ap.add_argument("--order", default="fig8", choices=["fig8", "eq5"],
                    help="main work of a mini-batch: forward O, update O, forward X, update X (the paper's Fig. 8, "
                         "default), or both forwards and then one update of every touched row (Eq. 5)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-hot-only", action="store_true", help="skip the hot-only section of the line")
    ap.add_argument("--blocks", type=int, default=10,
                    help="repetitions of the timed block of --steps steps, for the spread reported in `blocks`")
    ap.add_argument("--main-priority", type=int, default=-1,
                    help="CUDA priority of the main stream (forwards and updates); 0 = default, negative = higher")
    ap.add_argument("--index-priority", type=int, default=0,
                    help="CUDA priority of the streams of index-only ahead-work (fragment, cold-row search, sort)")
    ap.add_argument("--link-priority", type=int, default=0, help="CUDA priority of the host-link transfer streams")
    ap.add_argument("--mover-ctas", type=int, default=0, help="hl_set_mover_ctas: CTAs of the host reads (0 = default)")
    ap.add_argument("--scatter-ctas", type=int, default=0, help="hl_set_mover_ctas: CTAs of the write-backs")
    ap.add_argument("--write-back", choices=("overlap", "exclusive", "after_forward"), default="overlap",
                    help="hl_pipe_options.write_back: when a mini-batch's write-back runs")
    ap.add_argument("--fwd-ctas", type=int, default=0, help="hl_set_kernel_width: forward CTAs per multiprocessor")
    ap.add_argument("--bwd-ctas", type=int, default=0, help="hl_set_kernel_width: backward-sum CTAs per multiprocessor")
    ap.add_argument("--timeline", default=None,
                    help="write the per-stream timeline of three mini-batches of the traced pass to this text file")
    ap.add_argument("--micro", default=None, choices=["fwd", "bwd", "gather", "tracker", "wide"],
                    help="time one library call in isolation")
    ap.add_argument("--micro-dist", default="uniform", choices=["uniform", "zipf"])
    ap.add_argument("--micro-batch", type=int, default=16384)
    ap.add_argument("--micro-dim", type=int, default=64)
    ap.add_argument("--sweep", action="store_true", help="hot-budget (popular ratio) and batch-size sweeps")
    args = ap.parse_args()
    if args.sweep:
        run_sweep(args)
        return
    if args.micro == "tracker":
        run_micro_tracker(args)
        return
    if args.micro == "wide":
        run_micro_wide(args)
        return
    if args.micro == "gather":
        run_micro_gather(args)
        return
    if args.micro:
        run_micro(args)
        return
    if args.warmup < 3:
        log("[bench] warm-up raised to 3 steps")
        args.warmup = 3
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # not under a launcher: start the ranks here (one process per GPU, each re-running this command line)
        raise SystemExit(spawn_ranks(sys.argv[1:], args.gpus))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        run_reference(args, rank, world)
    else:
        run_cuda(args, rank, local_rank, world)


if __name__ == "__main__":
    main()

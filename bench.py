#!/usr/bin/env python
"""Benchmark of the whole decode-step hot path (cache lookup, mask build of the misses, mask
rows out, apply + greedy argmax, state advance) on synthetic workloads.

    python bench.py --gpus N --steps K --warmup W [--workload json_warm] [--impl reference]

One "step" is one wg_decode_step call over the whole batch.  Every step sees fresh logits:
a ring of R pristine logits buffers is generated once; a timed region of K steps runs in
chunks of at most R steps, each chunk bracketed by barrier + synchronize and CUDA events, and
the ring is restored from the pristine copies between chunks, outside the timed region.  A
region shorter than 50 ms is repeated (30 regions) and the median region is reported, with the
fastest and the slowest beside it.  With N > 1 ranks every rank runs its own batch (rows are
independent: no collective on the data path) and the time is the maximum over ranks; started
without a launcher, `--gpus N` starts its N ranks itself.

After the headline workload the default run adds short passes of the other workloads under the
key "workloads" (step time, rows/s, tokens checked/s, cache hit rate, roofline of the kernel that
dominates each).
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from wg_workloads import BY_NAME, flatten, has_structural_byte, make_logits, make_vocab  # noqa: E402

# dram__bytes_read.sum + dram__bytes_write.sum of ONE launch of the dominant kernel, taken with ncu
# on the same launch shape, together with the SHA-256 of the kernel source at the time of the
# capture: a figure is only reported while the kernels are still the ones that were measured.
NCU_TRAFFIC = {
    # workload: (bytes per launch, sha256 of paper_2507_16768_b200/csrc/wg_kernels.cuh)
    "json_warm": (223.6e6, "4a3397f6540f3b09c3e698b0c00a57864591e4688cd7313d43975ebac2e40f58"),            # 2.7 MB read + 220.9 MB written
    "html_warm_free_text": (400.3e6, "4a3397f6540f3b09c3e698b0c00a57864591e4688cd7313d43975ebac2e40f58"),  # 258.3 MB read + 142.0 MB written
}


def kernel_source_hash() -> str:
    import hashlib
    path = os.path.join(ROOT, "paper_2507_16768_b200", "csrc", "wg_kernels.cuh")
    with open(path, "rb") as f:
        return hashlib.sha256(f.read()).hexdigest()


def measured_traffic(workload: str, full_batch: bool):
    """The ncu DRAM traffic of the workload's dominant kernel, or None when there is no capture of
    the kernels as they are now."""
    entry = NCU_TRAFFIC.get(workload)
    if not entry or not full_batch or entry[1] != kernel_source_hash():
        return None
    return entry[0]


METRIC = "masked logit rows/s (mask build+apply)"
UNIT = "rows/s"
FALLBACK_HBM_GBS = 6650.0
N_SMS = 148
SHORT_REGION_MS = 50.0      # a timed region shorter than this is repeated
REPEATS = 30
# the secondary passes of the default run: (key, workload, options)
SECONDARY = [
    ("html_tiny", "html_tiny", {}),
    ("html_tiny_graph", "html_tiny", {"graph": True}),
    ("json_lookup", "json_lookup", {}),
    ("json_lookup_graph", "json_lookup", {"graph": True}),
    ("cold_templates", "cold_templates", {}),
    ("cold_templates_dedupe", "cold_templates", {"dedupe": True}),
    ("dynamic_snippets", "dynamic_snippets", {}),
    ("html_warm_free_text", "html_warm_free_text", {}),
]


def parse_args(argv=None):
    p = argparse.ArgumentParser()
    p.add_argument("--gpus", type=int, default=1)
    p.add_argument("--steps", type=int, default=1024)
    p.add_argument("--warmup", type=int, default=64)
    p.add_argument("--impl", default="ours", choices=["ours", "reference"])
    p.add_argument("--workload", default="json_warm", choices=sorted(BY_NAME))
    p.add_argument("--batch", type=int, default=0, help="override the workload's batch size")
    p.add_argument("--ring", type=int, default=0, help="distinct logits buffers (0 = auto)")
    p.add_argument("--steer", type=float, default=None,
                   help="bonus added to tokens holding a structural character")
    p.add_argument("--graph", action="store_true",
                   help="replay each step as a recorded CUDA graph (small batches)")
    p.add_argument("--separate", action="store_true",
                   help="call wg_build_masks / wg_apply_mask / wg_advance instead of wg_decode_step")
    p.add_argument("--steer-all", action="store_true",
                   help="steer every structural character (rows then dwell in free-text slots)")
    p.add_argument("--dedupe", action="store_true",
                   help="cache-off workloads: build each distinct (grammar, state) of a step once "
                        "(the cache is cleared before every step)")
    p.add_argument("--enum-size", type=int, default=0,
                   help="dynamic_snippets: names per enum (1000 = the configuration taken literally)")
    p.add_argument("--cache-mode", default="dense", choices=["dense", "compact"],
                   help="storage of cached masks: packed rows, or allows / denies entries")
    p.add_argument("--split", default="rows", choices=["rows", "vocab"],
                   help="with N > 1 ranks: every rank its own batch (weak scaling, no collective), "
                        "or every rank all rows and one slice of the vocabulary, with a MAX "
                        "all-reduce of the packed (logit, token) pairs each step (strong scaling)")
    p.add_argument("--no-workloads", action="store_true", help="skip the secondary passes")
    p.add_argument("--no-cpu-baseline", action="store_true")
    p.add_argument("--no-e2e", action="store_true")
    p.add_argument("--cpu-seconds", type=float, default=12.0)
    return p.parse_args(argv)


def default_steer(w) -> float:
    # the JSON grammars move through their states on plain N(0, 2) logits, and the free-text
    # workload is meant to dwell in its slots; templates with free-text slots need the bonus to
    # leave a slot within a run
    return 0.0 if w.name in ("json_lookup", "json_warm", "html_warm_free_text") else 6.0


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ---------------------------------------------------------------------------------------
# starting the ranks
# ---------------------------------------------------------------------------------------
def spawn_command(n: int, argv, port: int):
    """The launcher command that runs this file as `n` ranks on this node."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
            "--master-addr", "127.0.0.1", "--master-port", str(port),
            os.path.abspath(__file__)] + list(argv)


def free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def spawn_ranks(args, argv) -> int:
    """`--gpus N` without a launcher: start the N ranks (NCCL's own log level is left alone)."""
    if args.impl == "ours":
        import torch
        have = torch.cuda.device_count()
        if have < args.gpus:
            raise SystemExit(f"--gpus {args.gpus}: this node shows {have} CUDA device(s)")
    return subprocess.call(spawn_command(args.gpus, argv, free_port()), cwd=ROOT)


class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.path = tempfile.mktemp(prefix="wg_clocks_", suffix=".csv")
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(device_index), f"--query-gpu={self.QUERY}",
                 "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1]))
                    mx.append(float(f[2]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                      "sw_power_cap"), f[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)),
                       reasons=sorted(reasons), samples=len(sm))
        return out


# ---------------------------------------------------------------------------------------
# the CPU checker as a timed baseline (also the whole "--impl reference" arm)
# ---------------------------------------------------------------------------------------
class OracleRun:
    """Runs the path on the CPU checker over `rows` rows of the workload, as it stands."""

    def __init__(self, w, rows: int, steer: float):
        import oracle
        self.oracle = oracle
        self.w, self.rows, self.steer = w, rows, steer
        self.vocab = make_vocab(w.V, w.vocab_seed)
        self.bonus = has_structural_byte(self.vocab, w.steer_bytes)
        n_gram = len({w.grammar_of_row(r) for r in range(rows)})
        self.trees = {}
        for r in range(rows):
            g = w.grammar_of_row(r)
            if g not in self.trees:
                self.trees[g] = oracle.Tree(flatten(w.grammar(g)))
        assert len(self.trees) == n_gram
        self.row_tree = [self.trees[w.grammar_of_row(r)] for r in range(rows)]
        self.cursors = [t.start() for t in self.row_tree]
        self.threads = max(1, min(rows, oracle.max_threads()))
        self.step_no = 0

    def step(self) -> float:
        o, V = self.oracle, self.vocab.size
        logits = make_logits(self.rows, V, self.w.dtype, [self.w.vocab_seed, 777], self.step_no,
                             self.bonus, self.steer)
        t0 = time.perf_counter()
        masks = o.masks(self.row_tree, self.vocab, self.cursors, n_threads=self.threads)
        tokens = o.argmax(logits, masks, V)
        o.apply_mask(logits, masks, V, n_threads=self.threads)
        for r in range(self.rows):
            rc, cur = o.advance(self.row_tree[r], self.vocab, self.cursors[r], int(tokens[r]))
            if rc == 0:
                self.cursors[r] = self.row_tree[r].start() if cur == o.DONE else cur
        dt = time.perf_counter() - t0
        self.step_no += 1
        return dt


def cpu_baseline(w, steer: float, budget_s: float) -> dict:
    rows = min(w.batch, 32)
    run = OracleRun(w, rows, steer)
    first = run.step()
    n_steps = int(max(1, min(64, budget_s / max(first, 1e-3))))
    total = sum(run.step() for _ in range(n_steps))
    return {"value": rows * n_steps / total, "unit": UNIT, "cores": run.threads, "kind": "oracle",
            "sample": f"{rows} rows x {n_steps} steps of {w.name} (mask + argmax + apply + advance,"
                      f" no cache), after 1 untimed step"}


def run_reference(args, w, steer: float) -> None:
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    rows = min(w.batch, 32)
    probe = OracleRun(w, rows, steer)
    per_step = probe.step()
    # bound the whole run to about two minutes of CPU work
    budget = 120.0 / max(1, args.steps + args.warmup)
    if per_step > budget and rows > 1:
        rows = max(1, int(rows * budget / per_step))
    run = OracleRun(w, rows, steer)
    for _ in range(args.warmup):
        run.step()
    total = sum(run.step() for _ in range(args.steps))
    value = rows * args.steps / total
    sample = f"{rows} of {w.batch} rows per step of {w.name}, every step timed"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": w.dtype,
        "data": "synthetic",
        "config": {"workload": w.name, "V": w.V, "batch": w.batch, "rows_per_step": rows,
                   "logits": w.dtype, "steer": steer},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": run.threads, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------
# the CUDA path
# ---------------------------------------------------------------------------------------
class Dist:
    """World, rank and the barrier of this run."""

    def __init__(self, torch):
        self.torch = torch
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.rank = int(os.environ.get("RANK", "0"))
        self.local = int(os.environ.get("LOCAL_RANK", "0"))
        torch.cuda.set_device(self.local)
        if self.world > 1:
            import torch.distributed as dist
            dist.init_process_group("nccl", device_id=torch.device("cuda", self.local))
            self.dist = dist

    def barrier(self):
        if self.world > 1:
            self.dist.barrier()
        self.torch.cuda.synchronize()

    def close(self):
        if self.world > 1:
            self.dist.destroy_process_group()


def l2_copy_gbs(torch) -> float:
    """Read + write bandwidth of an in-place pass over 48 MB that stay in L2 (best of 20 runs of
    8 back-to-back passes; the launch gaps between passes are part of the time)."""
    a = torch.ones(12 << 20, dtype=torch.float32, device="cuda")
    best = 1e9
    for _ in range(20):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(8):
            a.neg_()
        e1.record()
        torch.cuda.synchronize()
        best = min(best, e0.elapsed_time(e1) / 8)
    return 2 * a.numel() * 4 / (best * 1e-3) / 1e9


class Workbench:
    """One workload set up on this rank's GPU: vocabulary, grammars, context, logits ring."""

    def __init__(self, wg, torch, D: Dist, w, *, steer, batch=0, ring=0, steps_hint=64,
                 cache_mode="dense", split="rows", steer_all=False, dedupe=False, graph=False,
                 separate=False, enum_size=0):
        from paper_2507_16768_b200.sharding import vocab_slices
        self.wg, self.torch, self.D, self.w = wg, torch, D, w
        self.steer, self.graph, self.separate, self.dedupe = steer, graph, separate, dedupe
        self.cache_mode, self.split = cache_mode, split
        B = self.B = batch or w.batch
        V = self.V = w.V
        self.tdtype = torch.bfloat16 if w.dtype == "bf16" else torch.float32
        self.esize = 2 if w.dtype == "bf16" else 4
        vocab = make_vocab(V, w.vocab_seed)
        self.dv = wg.Vocab(vocab.offsets, vocab.data, vocab.eos_id)
        self.by_vocab = split == "vocab"
        if self.by_vocab and (graph or separate or dedupe):
            raise SystemExit("--split vocab goes through wg_decode_step_shard only")
        self.v_begin, self.v_end = vocab_slices(V, D.world)[D.rank] if self.by_vocab else (0, V)
        self.Vs = max(self.v_end - self.v_begin, 1)          # logits columns this rank holds

        grammar_ids = sorted({w.grammar_of_row(r) for r in range(B)})
        if enum_size:
            from wg_workloads import grammars
            compiled = {g: wg.Grammar(flatten(grammars.dynamic_snippet_template(g, enum_size=enum_size)))
                        for g in grammar_ids}
        else:
            compiled = {g: wg.Grammar(flatten(w.grammar(g))) for g in grammar_ids}
        self.n_states = sum(c.n_states for c in compiled.values())
        self.use_cache = w.use_cache or dedupe
        # every state of every grammar, but never more rows than a run can visit
        capacity = min(self.n_states + 64, 1 << 16) if w.use_cache else (B if dedupe else 0)
        self.ctx = ctx = wg.Context(self.dv, capacity, B, wg.WG_CACHE_COMPACT
                                    if cache_mode == "compact" else wg.WG_CACHE_DENSE)
        gid_of = {g: ctx.add_grammar(c) for g, c in compiled.items()}
        if w.prewarm:
            for g in grammar_ids:
                ctx.cache_prewarm(gid_of[g])
        self.d_gid = torch.tensor([gid_of[w.grammar_of_row(r)] for r in range(B)],
                                  dtype=torch.int32, device="cuda")
        # a row that starts one step late sits in DONE first: it emits EOS and then restarts
        self.d_sid = torch.tensor([compiled[w.grammar_of_row(r)].done_state if w.row_delay(r) else
                                   compiled[w.grammar_of_row(r)].start_state for r in range(B)],
                                  dtype=torch.int32, device="cuda")
        self.d_mask = torch.zeros((B, self.dv.W), dtype=torch.int32, device="cuda")
        self.d_tok = torch.zeros(B, dtype=torch.int32, device="cuda")
        self.d_status = torch.zeros(B, dtype=torch.int32, device="cuda")
        self.flags = (wg.WG_USE_CACHE if self.use_cache else wg.WG_NO_CACHE) | wg.WG_RESTART_ON_DONE

        # ring of pristine logits, generated on the device (seeded); at most ~20 GB in all
        self.row_bytes = self.Vs * self.esize
        self.ring = ring or int(max(4, min(64, steps_hint, (20 << 30) // (B * self.row_bytes))))
        gen = torch.Generator(device="cuda")
        gen.manual_seed(1234 + (0 if self.by_vocab else 7919 * D.rank))  # one batch for all slices
        steer_bytes = b"" if steer_all else w.steer_bytes
        bonus = torch.from_numpy(has_structural_byte(vocab, steer_bytes)).cuda().to(torch.float32) * steer
        self.pristine = []
        for _ in range(self.ring):
            x = torch.randn((B, V), generator=gen, device="cuda", dtype=torch.float32) * 2.0
            if steer:
                x += bonus
            self.pristine.append(x[:, self.v_begin:self.v_begin + self.Vs].to(self.tdtype).contiguous())
            del x
        late = [r for r in range(B) if w.row_delay(r)]
        if late:
            # a late row sees, one step later, the logits of the row before it (its leader)
            late_idx = torch.tensor(late, device="cuda")
            for i in range(self.ring):
                self.pristine[i][late_idx] = self.pristine[i - 1][late_idx - 1]
        self.work = [torch.empty_like(p) for p in self.pristine]
        self.plan = wg.StepPlan(ctx, self.d_gid, self.d_sid, self.d_mask, self.d_tok, self.d_status,
                                self.flags)
        self.graphs = None
        if graph:
            # one recorded step per logits buffer of the ring (the recorded arguments are fixed)
            self.graphs = [wg.StepGraph(ctx, self.d_gid, self.d_sid, wbuf, self.d_mask, self.d_tok,
                                        self.d_status, self.flags) for wbuf in self.work]
        self.stream = torch.cuda.current_stream()
        self.ws = torch.empty(wg.wg_apply_workspace_bytes(B), dtype=torch.uint8, device="cuda")
        self.d_keys = torch.zeros(B, dtype=torch.int64, device="cuda")
        self.instrumented = False      # library events or counters on: graphs are not replayed

    def close(self):
        self.graphs = None
        self.plan = None
        self.ctx.close()
        self.dv.close()
        self.pristine = self.work = None
        self.torch.cuda.empty_cache()

    def step(self, i):
        wg, ring = self.wg, self.ring
        if self.dedupe:
            self.ctx.cache_clear()          # nothing carries over: only rows of one step share
        if self.by_vocab:
            from paper_2507_16768_b200.sharding import reduce_best_keys
            if self.v_end > self.v_begin:
                wg.wg_decode_step_shard(self.ctx, self.d_gid, self.d_sid, self.work[i % ring],
                                        self.d_mask, self.v_begin, self.v_end, self.d_keys,
                                        self.flags & wg.WG_NO_CACHE)
            else:
                self.d_keys.fill_(-(1 << 63))
            reduce_best_keys(self.d_keys)
            wg.wg_advance_keys(self.ctx, self.d_gid, self.d_sid, self.d_keys, self.d_tok,
                               self.d_status, self.flags & wg.WG_RESTART_ON_DONE)
        elif self.separate:
            # the same step through the individual entry points (7 launches instead of 4)
            wg.wg_build_masks(self.ctx, self.d_gid, self.d_sid, self.d_mask, self.flags & wg.WG_NO_CACHE)
            wg.wg_apply_mask(self.work[i % ring], self.d_mask, self.V, self.d_tok, self.ws)
            wg.wg_advance(self.ctx, self.d_gid, self.d_sid, self.d_tok, self.d_status,
                          self.flags & wg.WG_RESTART_ON_DONE)
        elif self.graphs is not None and not self.instrumented:
            self.graphs[i % ring].launch(self.stream)
        else:
            self.plan(self.work[i % ring])

    def region(self, n) -> float:
        """n steps in chunks of at most `ring`; the summed device time in ms."""
        torch = self.torch
        total, done = 0.0, 0
        while done < n:
            m = min(self.ring, n - done)
            for dst, src in zip(self.work, self.pristine):
                dst.copy_(src)
            self.D.barrier()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for i in range(m):
                self.step(i)
            e1.record()
            self.D.barrier()
            total += e0.elapsed_time(e1)
            done += m
        return total

    def measure(self, steps, warmup) -> dict:
        """Warm-up, the timed region(s), then the instrumented passes (per-kernel events, build
        work counters).  Times are this rank's; the caller takes the maximum over ranks."""
        from paper_2507_16768_b200.sharding import max_over_ranks
        wg, ctx = self.wg, self.ctx
        self.region(warmup)
        ctx.reset_stats()
        launches0 = wg.kernel_launch_count()
        t0 = time.perf_counter()
        regions = [max_over_ranks(self.region(steps), device="cuda")]
        launches = wg.kernel_launch_count() - launches0
        stats = ctx.stats()
        if regions[0] < SHORT_REGION_MS:
            regions += [max_over_ranks(self.region(steps), device="cuda") for _ in range(REPEATS - 1)]
        wall = time.perf_counter() - t0
        bad = int((self.d_status != 0).sum().item())
        # per-kernel durations: the same steps once more, now with the library recording CUDA
        # events around its kernels on the launching stream (the events sit between the kernels,
        # so this pass is kept out of the headline time)
        self.instrumented = True
        ctx.set_timing(True)
        before = ctx.stats()["masks_built"]
        self.region(min(steps, 4096))
        built_timed = ctx.stats()["masks_built"] - before
        kt = ctx.get_timing()
        ctx.set_timing(False)
        work = None
        if not self.w.prewarm:
            # what the build kernel had to do, from its counting variant over a few steps (decided
            # by the workload, not by this rank's counters: every rank must make the same calls)
            ctx.reset_stats()
            ctx.count_build_work(True)
            self.region(min(steps, 16))
            ctx.count_build_work(False)
            work = ctx.build_work()
            work["masks"] = ctx.stats()["masks_built"]
        self.instrumented = False
        ms = float(np.median(regions))
        out = {"ms": ms, "steps": steps, "regions_ms": regions, "launches": launches, "stats": stats,
               "bad": bad, "wall": wall,
               "apply_ms": kt["apply_ms"] / max(1, kt["steps"]),
               "build_ms": kt["build_ms"] / max(1, kt["steps"]),
               "built_per_timed_step": built_timed / max(1, kt["steps"]), "build_work": work}
        return out

    # ---- derived figures --------------------------------------------------------------
    def algorithmic_bytes(self) -> int:
        """Per step: every logit touched once, the cached mask read, the bitmask row written."""
        return self.B * (self.row_bytes + 2 * (self.Vs // 8))

    def roofline(self, m, peak, peak_kind, clocks, l2_gbs) -> dict:
        apply_ms, build_ms = m["apply_ms"], m["build_ms"]
        if self.w.use_cache or build_ms < apply_ms:
            algo = self.algorithmic_bytes()
            achieved = algo / (apply_ms * 1e-3) / 1e9 if apply_ms > 0 else 0.0
            step_gbs = algo / (m["ms"] / m["steps"] * 1e-3) / 1e9
            return {"kernel": "apply_mask_kernel (gather + apply + argmax)", "bound": "hbm",
                    "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                    "peak_kind": f"of {peak_kind}",
                    "traffic": measured_traffic(self.w.name, self.B == self.w.batch),
                    "algorithmic_bytes_per_launch": algo, "avg_launch_ms": apply_ms,
                    "whole_step": {"achieved": step_gbs, "frac": step_gbs / peak,
                                   "what": "the same bytes over the whole step's time"},
                    "timed_by": "CUDA events recorded by the library around the kernel, in a "
                                "second pass over the same steps"}
        # The build kernel: a bound from the work itself.  Per launch it must write the mask words
        # and read the vocabulary-mask words of its word-wise phase and a 16-byte record plus a
        # length byte per walked token, all through L2 (at the copy bandwidth of an L2-resident
        # buffer, measured in this run); and every table look-up of a walk is a gather that costs
        # one L1 pass, one per SM and clock.  The two do not overlap in this bound.
        work = m["build_work"] or {}
        masks = max(1, work.get("masks", 0))
        per_launch = m["built_per_timed_step"] / masks
        sm_hz = (clocks.get("sm_mhz") or 1965.0) * 1e6
        l2_bytes = per_launch * (4 * work.get("mask_words_read", 0) + 17 * work.get("tokens_walked", 0)) \
            + m["built_per_timed_step"] * 4 * (self.Vs // 32)
        lookups = per_launch * work.get("table_lookups", 0)
        bound_ms = (l2_bytes / (l2_gbs * 1e9) + lookups / (N_SMS * sm_hz)) * 1e3
        tok_per_s = m["built_per_timed_step"] * self.Vs / (build_ms * 1e-3) if build_ms > 0 else 0.0
        peak_tok = m["built_per_timed_step"] * self.Vs / (bound_ms * 1e-3) if bound_ms > 0 else 0.0
        return {"kernel": "build_masks_kernel (+ row reset)", "bound": "alu",
                "achieved": tok_per_s / 1e9, "peak": peak_tok / 1e9, "unit": "G tokens checked/s",
                "frac": tok_per_s / peak_tok if peak_tok else 0.0,
                "peak_kind": "derived from the work counted by the kernel: L2 bytes over the "
                             "measured L2 copy bandwidth plus table look-ups at one per SM and clock",
                "traffic": None, "avg_launch_ms": build_ms, "bound_ms": bound_ms,
                "l2_copy_gbs": l2_gbs,
                "per_mask": {"tokens_walked": work.get("tokens_walked", 0) / masks,
                             "table_lookups": work.get("table_lookups", 0) / masks,
                             "mask_words_read": work.get("mask_words_read", 0) / masks,
                             "words_written": self.Vs // 32}}

    def summary(self, m, peak, peak_kind, clocks, l2_gbs) -> dict:
        """The short record of a secondary pass."""
        world = 1 if self.by_vocab else self.D.world
        ms_step = m["ms"] / m["steps"]
        st = m["stats"]
        seen = st["cache_hits"] + st["cache_misses"]
        return {"workload": self.w.name, "V": self.V, "batch": self.B, "logits": self.w.dtype,
                "launch": "cuda graph" if self.graph else "stream",
                "cache": ("cleared every step (rows of one step share)" if self.dedupe else
                          "prewarmed" if self.w.prewarm else "on" if self.w.use_cache else "off"),
                "steer": self.steer, "states": self.n_states, "steps": m["steps"],
                "regions": len(m["regions_ms"]),
                "us_per_step": 1e3 * ms_step,
                "us_per_step_min_max": [1e3 * min(m["regions_ms"]) / m["steps"],
                                        1e3 * max(m["regions_ms"]) / m["steps"]],
                "rows_per_s": self.B * world / (ms_step * 1e-3),
                "masks_built_per_step": st["masks_built"] / m["steps"],
                "tokens_checked_per_s": st["masks_built"] * self.Vs / (m["regions_ms"][0] * 1e-3),
                "hit_rate": st["cache_hits"] / seen if seen else None,
                "cache_entries": st["cache_entries"], "cache_bytes": st["cache_bytes"],
                "kernel_us": {"lookup_and_build": 1e3 * m["build_ms"], "apply": 1e3 * m["apply_ms"]},
                "rows_with_error_status": m["bad"],
                "roofline": self.roofline(m, peak, peak_kind, clocks, l2_gbs)}


def run_e2e(bench: Workbench, n_steps: int):
    """The same metric through the host-buffer entry point: pinned host logits in, tokens out."""
    from paper_2507_16768_b200.sharding import max_over_ranks
    wg, torch, B = bench.wg, bench.torch, bench.B
    host_ring = [torch.empty((B, bench.V), dtype=bench.tdtype).pin_memory() for _ in range(2)]
    for h, p in zip(host_ring, bench.pristine):
        h.copy_(p)
    tok_host = torch.zeros(B, dtype=torch.int32).pin_memory()
    stage = bench.work[0]

    def one(i):
        wg.wg_decode_step_host(bench.ctx, bench.d_gid, bench.d_sid, host_ring[i % 2], stage,
                               bench.d_mask, bench.d_tok, tok_host, bench.d_status, bench.flags)
    for i in range(2):
        one(i)
    bench.D.barrier()
    t0 = time.perf_counter()
    for i in range(n_steps):
        one(i)
    bench.D.barrier()
    dt = max_over_ranks(time.perf_counter() - t0, device="cuda")
    return {"value": B * n_steps * bench.D.world / dt, "unit": UNIT,
            "h2d_bytes_per_step": B * bench.row_bytes, "d2h_bytes_per_step": 4 * B, "steps": n_steps}


def run_ours(args, w, steer: float) -> None:
    import torch

    from paper_2507_16768_b200 import build as lib_build
    if int(os.environ.get("LOCAL_RANK", "0")) == 0:
        lib_build.ensure()          # one rank builds if the library is missing
    import paper_2507_16768_b200 as wg

    D = Dist(torch)
    peak, peak_kind = measured_peak()
    bench = Workbench(wg, torch, D, w, steer=steer, batch=args.batch, ring=args.ring,
                      steps_hint=args.steps + args.warmup, cache_mode=args.cache_mode,
                      split=args.split, steer_all=args.steer_all, dedupe=args.dedupe,
                      graph=args.graph, separate=args.separate, enum_size=args.enum_size)
    sampler = ClockSampler(D.local) if D.rank == 0 else None
    m = bench.measure(args.steps, args.warmup)
    clocks = sampler.stop() if sampler else {}
    e2e = None
    if not args.no_e2e and not bench.by_vocab:
        e2e = run_e2e(bench, max(1, min(args.steps, 16)))
    l2_gbs = l2_copy_gbs(torch)

    if D.rank != 0:
        D.close()
        return
    by_vocab, B, V = bench.by_vocab, bench.B, bench.V
    stats = m["stats"]
    rows_total = B * args.steps * (1 if by_vocab else D.world)
    regions = m["regions_ms"]
    line = {
        "metric": METRIC, "value": rows_total / (m["ms"] * 1e-3), "unit": UNIT, "n_gpus": D.world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": m["ms"] / args.steps,
        "higher_is_better": True, "scaling": "strong" if by_vocab else "weak", "vs_baseline": None,
        "dtype": w.dtype, "data": "synthetic",
        "config": {"workload": w.name, "V": V, "batch_per_gpu": B, "logits": w.dtype,
                   "split": args.split, "vocab_slice": [bench.v_begin, bench.v_end],
                   "states": bench.n_states, "launch": "separate calls" if args.separate else
                   ("cuda graph" if args.graph else "stream"), "cache": "prewarmed" if w.prewarm else
                   ("on" if w.use_cache else ("cleared every step" if args.dedupe else "off")),
                   "cache_mode": args.cache_mode, "steer": steer, "ring": bench.ring,
                   "enum_size": args.enum_size or None,
                   "l2": "inputs larger than L2" if B * bench.row_bytes > (126 << 20) else
                   "ring of distinct buffers; working set may sit in L2",
                   "timing": f"CUDA events per chunk of <= ring steps, logits restored between "
                             f"chunks outside the timed region; {len(regions)} timed region(s) of "
                             f"{args.steps} steps, the median region reported"},
        "repeats": {"regions": len(regions), "ms_per_step_min": min(regions) / args.steps,
                    "ms_per_step_median": float(np.median(regions)) / args.steps,
                    "ms_per_step_max": max(regions) / args.steps},
        "roofline": bench.roofline(m, peak, peak_kind, clocks, l2_gbs),
        "kernel_ms": {"lookup_and_build": m["build_ms"], "apply": m["apply_ms"]},
        "tokens_checked_per_s": stats["masks_built"] * bench.Vs / (regions[0] * 1e-3),
        "cache": {k: stats[k] for k in ("cache_hits", "cache_misses", "masks_built",
                                         "rows_uncached", "cache_entries", "cache_bytes")},
        "rows_with_error_status": m["bad"],
        "e2e": e2e, "gpu_launches": m["launches"], "clocks": clocks, "wall_s": m["wall"],
    }
    bench.close()
    if D.world == 1 and not args.no_workloads and w.name == "json_warm" and not args.batch:
        line["workloads"] = secondary_passes(wg, torch, D, args, peak, peak_kind, clocks, l2_gbs)
    if not args.no_cpu_baseline and D.world == 1:
        line["cpu_baseline"] = cpu_baseline(w, steer, args.cpu_seconds)
    print(json.dumps(line), flush=True)
    D.close()


def secondary_passes(wg, torch, D, args, peak, peak_kind, clocks, l2_gbs) -> dict:
    """Short passes of the other workloads (N = 1 only): each its own set-up, 8 warm-up steps and
    timed regions of at most 128 steps."""
    out = {}
    for key, name, opts in SECONDARY:
        w = BY_NAME[name]
        steps = min(w.steps, 128)
        warm = 48 if name == "html_warm_free_text" else 8   # rows first walk into their slots
        try:
            b = Workbench(wg, torch, D, w, steer=default_steer(w), steps_hint=steps + warm,
                          cache_mode=args.cache_mode, **opts)
            out[key] = b.summary(b.measure(steps, warm), peak, peak_kind, clocks, l2_gbs)
            b.close()
        except Exception as e:          # a failed secondary pass must not lose the headline
            out[key] = {"error": f"{type(e).__name__}: {e}"}
    return out


def main():
    argv = sys.argv[1:]
    args = parse_args(argv)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        raise SystemExit(spawn_ranks(args, argv))
    w = BY_NAME[args.workload]
    steer = default_steer(w) if args.steer is None else args.steer
    if args.impl == "reference":
        run_reference(args, w, steer)
    else:
        run_ours(args, w, steer)


if __name__ == "__main__":
    main()

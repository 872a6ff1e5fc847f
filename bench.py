#!/usr/bin/env python
"""Benchmark of the whole decode-step hot path (cache lookup, mask build of the misses, mask
rows out, apply + greedy argmax, state advance) on synthetic workloads.

    python bench.py --gpus 1 --steps K --warmup W [--workload json_warm] [--impl reference]

One "step" is one wg_decode_step call over the whole batch.  Every step sees fresh logits:
a ring of R pristine logits buffers is generated once; the timed region runs in chunks of at
most R steps, each chunk bracketed by barrier + synchronize and CUDA events, and the ring is
restored from the pristine copies between chunks, outside the timed region.  With N > 1
ranks every rank runs its own batch (rows are independent: no collective on the data path)
and the time is the maximum over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from wg_workloads import BY_NAME, flatten, has_structural_byte, make_logits, make_vocab  # noqa: E402

# dram__bytes_read.sum + dram__bytes_write.sum of ONE launch of the dominant kernel, from the ncu
# capture summarised under profiles/ (same launch shape as the timed run).  Set an entry to None
# when its kernel changes and the capture has not been redone.
BUILD_WARP_INSTR_PER_TOKEN = 0.44  # mean of the two launches under profiles/build_masks_kernel_cold_templates*.md

NCU_TRAFFIC_BYTES = {
    "json_warm": 220.9e6,       # profiles/apply_mask_kernel_json_warm.md
}
# the build kernel reads vocabulary masks, token records and tables that sit in L2: DRAM reads of
# one launch, mean of the early and the late step under profiles/build_masks_kernel_cold_templates*.md
NCU_BUILD_TRAFFIC_BYTES = {
    "cold_templates": 5.7e6,
}

METRIC = "masked logit rows/s (mask build+apply)"
UNIT = "rows/s"
FALLBACK_HBM_GBS = 6650.0


def parse_args():
    p = argparse.ArgumentParser()
    p.add_argument("--gpus", type=int, default=1)
    p.add_argument("--steps", type=int, default=2048)
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
    p.add_argument("--cache-mode", default="dense", choices=["dense", "compact"],
                   help="storage of cached masks: packed rows, or allows / denies entries")
    p.add_argument("--split", default="rows", choices=["rows", "vocab"],
                   help="with N > 1 ranks: every rank its own batch (weak scaling, no collective), "
                        "or every rank all rows and one slice of the vocabulary, with a MAX "
                        "all-reduce of the packed (logit, token) pairs each step (strong scaling)")
    p.add_argument("--no-cpu-baseline", action="store_true")
    p.add_argument("--no-e2e", action="store_true")
    p.add_argument("--cpu-seconds", type=float, default=12.0)
    return p.parse_args()


def default_steer(w) -> float:
    # the JSON grammars move through their states on plain N(0, 2) logits; templates with
    # free-text slots need the bonus to leave a slot within a run
    return 0.0 if w.name in ("json_lookup", "json_warm") else 6.0


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


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
                 "--format=csv,noheader,nounits", "-lms", "50"],
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
def run_ours(args, w, steer: float) -> None:
    import torch
    import torch.distributed as dist

    from paper_2507_16768_b200 import build as lib_build
    if int(os.environ.get("LOCAL_RANK", "0")) == 0:
        lib_build.ensure()          # one rank builds if the library is missing
    import paper_2507_16768_b200 as wg
    from paper_2507_16768_b200.sharding import max_over_ranks

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    B = args.batch or w.batch
    V = w.V
    tdtype = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    esize = 2 if w.dtype == "bf16" else 4
    vocab = make_vocab(V, w.vocab_seed)
    dv = wg.Vocab(vocab.offsets, vocab.data, vocab.eos_id)
    W = dv.W

    by_vocab = args.split == "vocab"
    if by_vocab and (args.graph or args.separate):
        raise SystemExit("--split vocab goes through wg_decode_step_shard only")
    from paper_2507_16768_b200.sharding import reduce_best_keys, vocab_slices
    v_begin, v_end = vocab_slices(V, world)[rank] if by_vocab else (0, V)
    Vs = max(v_end - v_begin, 1)          # logits columns this rank holds

    grammar_ids = sorted({w.grammar_of_row(r) for r in range(B)})
    compiled = {g: wg.Grammar(flatten(w.grammar(g))) for g in grammar_ids}
    n_states = sum(c.n_states for c in compiled.values())
    # every state of every grammar, but never more rows than a run can visit
    capacity = min(n_states + 64, 1 << 16) if w.use_cache else 0
    ctx = wg.Context(dv, capacity, B, wg.WG_CACHE_COMPACT if args.cache_mode == "compact"
                     else wg.WG_CACHE_DENSE)
    gid_of = {g: ctx.add_grammar(c) for g, c in compiled.items()}
    if w.prewarm:
        for g in grammar_ids:
            ctx.cache_prewarm(gid_of[g])
    d_gid = torch.tensor([gid_of[w.grammar_of_row(r)] for r in range(B)], dtype=torch.int32,
                         device="cuda")
    # a row that starts one step late sits in DONE first: it emits EOS and then restarts
    d_sid = torch.tensor([compiled[w.grammar_of_row(r)].done_state if w.row_delay(r) else
                          compiled[w.grammar_of_row(r)].start_state for r in range(B)],
                         dtype=torch.int32, device="cuda")
    d_mask = torch.zeros((B, W), dtype=torch.int32, device="cuda")
    d_tok = torch.zeros(B, dtype=torch.int32, device="cuda")
    d_status = torch.zeros(B, dtype=torch.int32, device="cuda")
    flags = (wg.WG_USE_CACHE if w.use_cache else wg.WG_NO_CACHE) | wg.WG_RESTART_ON_DONE

    # ring of pristine logits, generated on the device (seeded); at most ~40 GB in all
    row_bytes = Vs * esize
    ring = args.ring or int(max(4, min(64, args.steps + args.warmup, (20 << 30) // (B * row_bytes))))
    gen = torch.Generator(device="cuda")
    gen.manual_seed(1234 + (0 if by_vocab else 7919 * rank))   # one batch for all vocabulary slices
    steer_bytes = b"" if args.steer_all else w.steer_bytes
    bonus = torch.from_numpy(has_structural_byte(vocab, steer_bytes)).cuda().to(torch.float32) * steer
    pristine = []
    for _ in range(ring):
        x = torch.randn((B, V), generator=gen, device="cuda", dtype=torch.float32) * 2.0
        if steer:
            x += bonus
        pristine.append(x[:, v_begin:v_begin + Vs].to(tdtype).contiguous())
        del x
    late = [r for r in range(B) if w.row_delay(r)]
    if late:
        # a late row sees, one step later, the logits of the row before it (its leader)
        late_idx = torch.tensor(late, device="cuda")
        for i in range(ring):
            pristine[i][late_idx] = pristine[i - 1][late_idx - 1]
    work = [torch.empty_like(p) for p in pristine]

    timing_pass = [False]

    def restore():
        for dst, src in zip(work, pristine):
            dst.copy_(src)

    plan = wg.StepPlan(ctx, d_gid, d_sid, d_mask, d_tok, d_status, flags)
    graphs = None
    if args.graph:
        # one recorded step per logits buffer of the ring (the recorded arguments are fixed)
        graphs = [wg.StepGraph(ctx, d_gid, d_sid, wbuf, d_mask, d_tok, d_status, flags)
                  for wbuf in work]
        stream_ptr = torch.cuda.current_stream()

    ws = torch.empty(wg.wg_apply_workspace_bytes(B), dtype=torch.uint8, device="cuda")

    d_keys = torch.zeros(B, dtype=torch.int64, device="cuda")

    def step(i):
        if by_vocab:
            if v_end > v_begin:
                wg.wg_decode_step_shard(ctx, d_gid, d_sid, work[i % ring], d_mask, v_begin, v_end,
                                        d_keys, flags & wg.WG_NO_CACHE)
            else:
                d_keys.fill_(-(1 << 63))
            reduce_best_keys(d_keys)
            wg.wg_advance_keys(ctx, d_gid, d_sid, d_keys, d_tok, d_status,
                               flags & wg.WG_RESTART_ON_DONE)
        elif args.separate:
            # the same step through the individual entry points (7 launches instead of 4)
            wg.wg_build_masks(ctx, d_gid, d_sid, d_mask, flags & wg.WG_NO_CACHE)
            wg.wg_apply_mask(work[i % ring], d_mask, V, d_tok, ws)
            wg.wg_advance(ctx, d_gid, d_sid, d_tok, d_status, flags & wg.WG_RESTART_ON_DONE)
        elif graphs is not None and not timing_pass[0]:
            graphs[i % ring].launch(stream_ptr)
        else:
            plan(work[i % ring])

    def run_steps(n, timed):
        """n steps in chunks of at most `ring`; returns the summed device time in ms."""
        total, done = 0.0, 0
        while done < n:
            m = min(ring, n - done)
            restore()
            barrier()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for i in range(m):
                step(i)
            e1.record()
            barrier()
            total += e0.elapsed_time(e1)
            done += m
        return total

    run_steps(args.warmup, False)
    ctx.reset_stats()
    sampler = ClockSampler(local) if rank == 0 else None
    launches0 = wg.kernel_launch_count()
    t_wall0 = time.perf_counter()
    ms = run_steps(args.steps, True)
    wall = time.perf_counter() - t_wall0
    launches = wg.kernel_launch_count() - launches0
    stats = ctx.stats()
    bad = int((d_status != 0).sum().item())
    # per-kernel durations: the same steps once more, now with the library recording CUDA
    # events around its kernels on the launching stream (the events sit between the kernels,
    # so this pass is kept out of the headline time)
    ctx.set_timing(True)
    timing_pass[0] = True
    kernel_pass_ms = run_steps(min(args.steps, 4096), True)
    built_timed = ctx.stats()["masks_built"] - stats["masks_built"]
    kt = ctx.get_timing()
    ctx.set_timing(False)
    clocks = sampler.stop() if sampler else {}

    ms = max_over_ranks(ms, device="cuda")
    rows_total = B * args.steps * (1 if by_vocab else world)
    value = rows_total / (ms * 1e-3)

    # ---- end to end through the host-buffer entry point: pinned host logits in, tokens out
    e2e = None
    if not args.no_e2e and not by_vocab:
        n_e2e = max(1, min(args.steps, 16))
        host_ring = [torch.empty((B, V), dtype=tdtype).pin_memory() for _ in range(2)]
        for h, p in zip(host_ring, pristine):
            h.copy_(p)
        tok_host = torch.zeros(B, dtype=torch.int32).pin_memory()
        stage = work[0]
        for i in range(2):
            wg.wg_decode_step_host(ctx, d_gid, d_sid, host_ring[i % 2], stage, d_mask, d_tok,
                                   tok_host, d_status, flags)
        barrier()
        t0 = time.perf_counter()
        for i in range(n_e2e):
            wg.wg_decode_step_host(ctx, d_gid, d_sid, host_ring[i % 2], stage, d_mask, d_tok,
                                   tok_host, d_status, flags)
        barrier()
        dt = time.perf_counter() - t0
        dt = max_over_ranks(dt, device="cuda")
        e2e = {"value": B * n_e2e * world / dt, "unit": UNIT, "h2d_bytes_per_step": B * row_bytes,
               "d2h_bytes_per_step": 4 * B, "steps": n_e2e}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_peak()
    algo_bytes = B * (row_bytes + 2 * (Vs // 8))
    apply_ms = kt["apply_ms"] / max(1, kt["steps"])
    build_ms = kt["build_ms"] / max(1, kt["steps"])
    built = stats["masks_built"]
    del kernel_pass_ms
    if w.use_cache or build_ms < apply_ms:
        achieved = algo_bytes / (apply_ms * 1e-3) / 1e9 if apply_ms > 0 else 0.0
        roofline = {"kernel": "apply_mask_kernel (gather + apply + argmax)", "bound": "hbm",
                    "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                    "peak_kind": f"of {peak_kind}",
                    "traffic": NCU_TRAFFIC_BYTES.get(w.name) if B == w.batch else None,
                    "algorithmic_bytes_per_launch": algo_bytes, "avg_launch_ms": apply_ms,
                    "timed_by": "CUDA events recorded by the library around the kernel, in a "
                                "second pass over the same steps"}
    else:
        # Issue-slot bound of the build kernel: 148 SMs x 4 schedulers x 1 warp instruction per
        # clock at the sampled SM clock, divided by the warp instructions the kernel spends per
        # token checked (ncu: 13.8 M and 20.2 M instructions for two launches of 256 x 151 936
        # tokens, early and late in a run: 0.44 per token on average).
        sm_mhz = clocks.get("sm_mhz") or 1965.0
        peak_tok = 148 * 4 * sm_mhz * 1e6 / BUILD_WARP_INSTR_PER_TOKEN
        tok_per_s = built_timed * Vs / (kt["build_ms"] * 1e-3) if kt["build_ms"] > 0 else 0.0
        roofline = {"kernel": "build_masks_kernel (+ row reset)", "bound": "alu",
                    "achieved": tok_per_s / 1e9, "peak": peak_tok / 1e9,
                    "unit": "G tokens checked/s", "frac": tok_per_s / peak_tok,
                    "peak_kind": "issue slots at the kernel's measured instructions per token",
                    "traffic": NCU_BUILD_TRAFFIC_BYTES.get(w.name) if B == w.batch else None,
                    "avg_launch_ms": build_ms}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True,
        "scaling": "strong" if by_vocab else "weak", "vs_baseline": None, "dtype": w.dtype,
        "data": "synthetic",
        "config": {"workload": w.name, "V": V, "batch_per_gpu": B, "logits": w.dtype,
                   "split": args.split, "vocab_slice": [v_begin, v_end],
                   "states": n_states, "launch": "separate calls" if args.separate else
                   ("cuda graph" if args.graph else "stream"), "cache": "prewarmed" if w.prewarm else
                   ("on" if w.use_cache else "off"), "cache_mode": args.cache_mode, "steer": steer,
                   "ring": ring,
                   "l2": "inputs larger than L2" if B * row_bytes > (126 << 20) else
                   "ring of distinct buffers; working set may sit in L2",
                   "timing": "CUDA events per chunk of <= ring steps; logits restored between "
                             "chunks outside the timed region"},
        "roofline": roofline,
        "kernel_ms": {"lookup_and_build": build_ms, "apply": apply_ms},
        "tokens_checked_per_s": (built * Vs) / (ms * 1e-3) if built else 0.0,
        "cache": {k: stats[k] for k in ("cache_hits", "cache_misses", "masks_built",
                                         "rows_uncached", "cache_entries", "cache_bytes")},
        "rows_with_error_status": bad,
        "e2e": e2e, "gpu_launches": launches, "clocks": clocks, "wall_s": wall,
    }
    if not args.no_cpu_baseline and world == 1:
        line["cpu_baseline"] = cpu_baseline(w, steer, args.cpu_seconds)
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    args = parse_args()
    w = BY_NAME[args.workload]
    steer = default_steer(w) if args.steer is None else args.steer
    if args.impl == "reference":
        run_reference(args, w, steer)
    else:
        run_ours(args, w, steer)


if __name__ == "__main__":
    main()

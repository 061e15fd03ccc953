"""Sensitivity sweeps of the rebalancer on the synthetic workloads (paper Section 4.5):
migration_batch_size B in {1 .. 256} (stage 1) and the threshold pairs (stage 2), plus the
static partition and the default cell with the reclaim_gap variant of the waste rule, reporting the event-deterministic fields the paper tabulates -- OOM count,
rebalance events, migrated MiB -- and, because this build really moves payload, relocated MiB
and the device time spent relocating.

    python -m paper_2605_22416_b200.sweep --workload short_uniform --steps 3000

Every cell is a closed-loop run through the C ABI on the GPU (`avmp_step_host` per engine
step).  `run_cell` takes the engine as an argument so tests can run the same cell against
another implementation and compare.
"""
from __future__ import annotations

import argparse
import json
from typing import Callable, Dict, List, Optional

import numpy as np

from . import workloads as W

B_VALUES = (1, 2, 4, 8, 16, 32, 64, 128, 256)
THRESHOLDS = ((50_000, 300_000), (20_000, 300_000), (100_000, 300_000), (50_000, 100_000), (50_000, 200_000))


def run_cell(w: W.Workload, step_fn: Callable[[np.ndarray], np.ndarray], stats_fn: Callable[[], dict],
             steps: int) -> Dict:
    """One closed-loop run of `steps` engine steps; returns the event-deterministic summary."""
    trace, d = W.record_trace(w, step_fn, max_steps=steps)
    s = stats_fn()
    return {
        "B": w.migration_batch_size, "th_low": w.threshold_low_ppm / 1e6, "th_high": w.threshold_high_ppm / 1e6,
        "dynamic": bool(w.migration_enabled), "reclaim_gap": bool(w.reclaim_gap), "steps": d.step, "ops": s["op_counter"], "n_oom": s["n_oom"],
        "rebalances": s["n_rebalance"], "migrated_mib": s["migrated_bytes"] / W.MiB,
        "relocated_mib": s["relocated_bytes"] / W.MiB, "wasted_kib": s["wasted_bytes"] / 1024,
        "relocation_ms": s.get("relocation_ns_total", 0) / 1e6,
        "oom_retry_share": s.get("step_ns_oom_retry", 0) / max(s.get("step_ns_total", 0), 1),
        "migration_plan_share": s.get("step_ns_migration_plan", 0) / max(s.get("step_ns_total", 0), 1),
        "completed": d.completed,
        "preempted": d.preempted, "cap_kv": s["cap_kv"], "cap_ssm": s["cap_ssm"],
    }


def cells(base: W.Workload, stage: str) -> List[W.Workload]:
    out = [base.with_(migration_enabled=False)]
    if stage in ("b", "all"):
        out += [base.with_(migration_batch_size=b) for b in B_VALUES]
    if stage in ("thresholds", "all"):
        out += [base.with_(threshold_low_ppm=lo, threshold_high_ppm=hi) for lo, hi in THRESHOLDS]
    out.append(base.with_(reclaim_gap=True))
    return out


def gpu_cell(w: W.Workload, steps: int, device="cuda:0") -> Dict:
    from . import binding as B
    ctx = B.Context.from_workload(w, device=device)

    def step_fn(ops: np.ndarray) -> np.ndarray:
        st = np.zeros(len(ops), np.uint32)
        ctx.step_host(np.ascontiguousarray(ops), len(ops), st)
        return st

    try:
        return run_cell(w, step_fn, ctx.stats, steps)
    finally:
        ctx.close()


def to_markdown(rows: List[Dict]) -> str:
    cols = ("dynamic", "reclaim_gap", "B", "th_low", "th_high", "n_oom", "rebalances", "migrated_mib", "relocated_mib",
            "relocation_ms", "oom_retry_share", "migration_plan_share", "completed", "preempted", "cap_kv", "cap_ssm")
    lines = ["| " + " | ".join(cols) + " |", "|" + "---|" * len(cols)]
    for r in rows:
        lines.append("| " + " | ".join(f"{r[c]:.2f}" if isinstance(r[c], float) else str(r[c]) for c in cols) + " |")
    return "\n".join(lines)


def main(argv: Optional[List[str]] = None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="short_uniform")
    ap.add_argument("--steps", type=int, default=3000)
    ap.add_argument("--stage", default="all", choices=["b", "thresholds", "all"])
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--json", action="store_true")
    args = ap.parse_args(argv)
    base = W.config(args.workload, seed=args.seed)
    rows = [gpu_cell(w, args.steps) for w in cells(base, args.stage)]
    print(json.dumps(rows) if args.json else f"### {args.workload}, {args.steps} steps, seed {args.seed}\n\n" + to_markdown(rows))


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the AVMP hot path on B200.

One "step" = one engine step of the whole path on one batch of the closed-loop trace:
avmp_step (admit / extend / finish batch, CapacityError handler, migration + relocation
copy), avmp_translate of every live handle of the running batch, avmp_gather_kv for every
attention layer and avmp_gather_ssm for every SSM layer of the running batch.

Workload of the headline: `scale`, the largest single-GPU configuration (72-layer hybrid, 9
attention + 63 Mamba layers, 120 GiB pool resident in HBM, split 0.5, B = 128, step batch
1024), synthetic and seeded.  The trace is produced closed loop against the library itself
(untimed), then replayed from device-resident op batches for the timed region.  Inputs exceed
L2: every step reads and writes about 190 GB.  The other four configurations are measured
the same way, briefly, and reported under roofline.other_configs.

Prints ONE JSON line: headline value, roofline of the dominant kernel (with the secondary
figures of the metric: KV gather, relocation copy, single-layer launches, allocator rate),
end-to-end figure, CPU baseline.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

from paper_2605_22416_b200 import workloads as W  # noqa: E402

METRIC = "paged gather+migration GB/s over whole engine steps (allocator ops/s reported beside it)"
WARM_STEPS = 600          # closed-loop steps before the measured window (steady state)
# DRAM traffic of one launch of the dominant kernel, from ncu captures of this kernel at 1 GB and at 6.8 GB per
# launch (summarised under profiles/):
# reads equal the algorithmic read bytes, and of the writes about 47 MB are still dirty in L2 when the kernel
# ends (they reach DRAM during the next kernel).  Recorded from those captures, not re-measured per run.
L2_DIRTY_TAIL_BYTES = 47e6
# timed steps and warm steps of the brief runs of the other configurations: each timed region exceeds 0.2 s
OTHER_CONFIGS = {"pr1": (2600, 400), "short_uniform": (200, 600), "mixed_long": (420, 600), "agentic_burst": (130, 600)}


def _peaks():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        return float(json.loads(p.read_text())["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


# ---------------------------------------------------------------------------------------
# clocks during the timed region (NVML, read-only)
# ---------------------------------------------------------------------------------------
class ClockSampler:
    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
               0x4: "sw_power_cap", 0x80: "hw_power_brake_slowdown"}

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._t = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                r = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                for bit, name in self.REASONS.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(0.02)

    def start(self):
        if self.nv is not None:
            self._t = threading.Thread(target=self._run, daemon=True)
            self._t.start()

    def stop(self) -> dict:
        self._stop.set()
        if self._t is not None:
            self._t.join()
        med = int(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# ---------------------------------------------------------------------------------------
# bytes moved by one step, by definition of the operations (not by counting kernel traffic)
# ---------------------------------------------------------------------------------------
def step_bytes(model: W.ModelShape, n_running: int, total_tokens: int, relocated_bytes: int) -> dict:
    kv = 2 * total_tokens * 2 * model.kv_row_bytes * model.n_attn_layers          # K and V, read + write
    ssm = 2 * n_running * (model.state_bytes + model.conv_bytes) * model.n_ssm_layers
    return {"kv": kv, "ssm": ssm, "reloc": 2 * relocated_bytes}


def config_dict(w: W.Workload, warm_steps: int = WARM_STEPS) -> dict:
    """What the workload is (the same dict for both arms; what a run saw goes under `workload_stats`)."""
    m = w.model
    return {"workload": w.name, "cache_shape": f"{m.n_attn_layers} attention + {m.n_ssm_layers} mamba layers, "
                                               f"KV page {m.page_tokens} tok x {m.kv_heads} x {m.head_dim} bf16, "
                                               f"SSM block {m.ssm_state_elems} + {m.ssm_conv_elems} fp32",
            "pool_gib": w.pool_bytes / W.GiB,
            "split": w.split, "migration_batch_size": w.migration_batch_size, "step_batch": w.concurrency,
            "warm_steps": warm_steps, "seed": w.seed,
            "l2": "inputs larger than L2: every launch reads its bytes from a multi-GiB arena for the first time in "
                  "the step and writes a batch buffer that the next group or step overwrites only after far more "
                  "than L2's 126 MB has passed through",
            "multi_gpu": "replicas only: one independent context per GPU, no collective"}


def reduce_over_ranks(local_ms: float, local_sums: np.ndarray, world: int):
    """max of the time, sum of the additive quantities, over all ranks (identity at world 1)."""
    if world == 1:
        return local_ms, local_sums
    import torch
    import torch.distributed as dist
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([local_ms], dtype=torch.float64, device=dev)
    s = torch.tensor(local_sums, dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(s, op=dist.ReduceOp.SUM)
    return float(t.item()), s.cpu().numpy()


def layers_per_launch(w: W.Workload, dev, max_run: int, max_tok: int, asked: int):
    """How many layers of batch buffers fit beside the arena: all attention layers, and as many SSM layers
    as the free memory holds (the launches of a step then walk the layers in groups of that size)."""
    import torch
    m = w.model
    if asked:
        return min(m.n_attn_layers, asked), min(m.n_ssm_layers, asked)
    free, _ = torch.cuda.mem_get_info(dev)
    free -= 6 * W.GiB                                            # tables, traces, slack
    kv_layer = 2 * max_tok * m.kv_row_bytes
    lpl_kv = int(max(1, min(m.n_attn_layers, (free // 2) // max(kv_layer, 1))))
    free -= lpl_kv * kv_layer
    ssm_layer = max_run * (m.state_bytes + m.conv_bytes)
    lpl_ssm = int(max(1, min(m.n_ssm_layers, free // max(ssm_layer, 1))))
    return lpl_kv, lpl_ssm


# ---------------------------------------------------------------------------------------
# our arm
# ---------------------------------------------------------------------------------------
def measure(w: W.Workload, dev, *, steps: int, warmup: int, warm_steps: int, asked_lpl: int, full: bool,
            world: int = 1) -> dict:
    """The hot path on one workload: K whole engine steps under one event pair, then the same window with an
    event pair per kernel class.  full: also one launch per layer, and the end-to-end loop with host buffers."""
    import torch
    from paper_2605_22416_b200 import binding as B

    m = w.model
    WS = warm_steps
    n_steps = WS + warmup + steps

    # ---- phase A: closed loop against the library (untimed) -> per-step batches ----
    ctx = B.Context.from_workload(w, device=dev)
    drv = W.ClosedLoopDriver(w, requests=W.make_requests(w, min(w.n_requests, 400 * w.concurrency))
                             if w.kind == "queue" else None)
    trace = []

    def held_units():
        # units every slot holds, from the driver's bookkeeping: pages of the chain, SSM blocks while running
        return -(-drv.len // m.page_tokens), np.where(drv.state == 1, m.n_ssm_layers, 0)

    while not drv.done and drv.step < n_steps:
        ops = drv.next_batch()
        st = np.zeros(len(ops), np.uint32)
        pages0, blocks0 = held_units()
        ctx.step_host(np.ascontiguousarray(ops), len(ops), st)
        drv.feed(st)
        pages1, blocks1 = held_units()
        rec = {"ops": ops, "run": drv.running_slots.astype(np.uint32), "lens": drv.len[drv.running_slots].copy(),
               # lower bound on units allocated + freed by this batch (a slot freed and re-admitted in one
               # step counts its net change only)
               "units": int(np.abs(pages1 - pages0).sum() + np.abs(blocks1 - blocks0).sum())}
        if drv.step > WS:
            t, _ = ctx.export_tables()
            chain = t["req_chain"].reshape(w.max_requests, w.max_pages)
            ssm = t["req_ssm"].reshape(w.max_requests, m.n_ssm_layers)
            rec["handles"] = np.concatenate([chain[r, :t["req_npages"][r]] for r in rec["run"]] +
                                            [ssm[rec["run"]].reshape(-1)]).astype(np.uint32)
        trace.append(rec)
    assert len(trace) == n_steps, f"{w.name}: trace ended after {len(trace)} of {n_steps} steps"
    stats_a = ctx.stats()
    arena = ctx.arena
    ctx.close()

    # ---- phase B: replay from device-resident batches ----
    stream = torch.cuda.current_stream()
    sid = stream.cuda_stream          # raw cudaStream_t, passed straight to the C ABI
    max_run = max(max(len(r["run"]) for r in trace[WS:]), 1)
    max_tok = max(max(int(r["lens"].sum()) for r in trace[WS:]), 1)
    max_h = max(max(len(r["handles"]) for r in trace[WS:]), 1)
    lpl_kv, lpl_ssm = layers_per_launch(w, dev, max_run, max_tok, asked_lpl)
    d_status = torch.zeros(w.concurrency * 2 + 16, dtype=torch.int32, device=dev)
    # batch buffers: one slab per kind, [layer][row]; the layers of a launch have their own rows (no reuse
    # inside a launch; the next group of layers reuses the slab)
    out_k = torch.empty((lpl_kv, max_tok, m.kv_row_bytes), dtype=torch.uint8, device=dev)
    out_v = torch.empty((lpl_kv, max_tok, m.kv_row_bytes), dtype=torch.uint8, device=dev)
    out_s = torch.empty((lpl_ssm, max_run, m.state_bytes), dtype=torch.uint8, device=dev)
    out_c = torch.empty((lpl_ssm, max_run, m.conv_bytes), dtype=torch.uint8, device=dev)
    kv_groups = [(f, min(lpl_kv, m.n_attn_layers - f)) for f in range(0, m.n_attn_layers, lpl_kv)]
    ssm_groups = [(f, min(lpl_ssm, m.n_ssm_layers - f)) for f in range(0, m.n_ssm_layers, lpl_ssm)]
    kv_stride, s_stride, c_stride = max_tok * m.kv_row_bytes, max_run * m.state_bytes, max_run * m.conv_bytes
    d_cu = torch.zeros(max_run + 1, dtype=torch.int32, device=dev)
    d_pool = torch.zeros(max_h, dtype=torch.int32, device=dev)
    d_off = torch.zeros(max_h, dtype=torch.int64, device=dev)
    d_aoff = torch.zeros(max_h, dtype=torch.int64, device=dev)

    def to_dev(a):
        a = np.ascontiguousarray(a)
        return torch.from_numpy(a.view(np.uint8).reshape(-1)).to(dev) if a.size else torch.zeros(16, dtype=torch.uint8, device=dev)

    for r in trace:
        r["d_ops"] = to_dev(r["ops"])
    for r in trace[WS:]:
        r["d_run"] = to_dev(r["run"])
        r["d_handles"] = to_dev(r["handles"])

    def ev():
        return torch.cuda.Event(enable_timing=True)

    # when the batch buffers of all layers fit, a step's payload moves in ONE launch (avmp_gather_step)
    one_launch = len(kv_groups) == 1 and len(ssm_groups) == 1

    def full_step(c, r, marks=None, per_layer=False, fused=False, separate_calls=False):
        """One engine step.  marks: one event pair per kernel class (allocator, KV, SSM).
        per_layer: one launch per layer instead of one launch per group of layers.
        fused: both gathers of all layers in one launch (the KV mark then coincides with the allocator mark)."""
        n_ops, n_run = len(r["ops"]), len(r["run"])
        cap_tok = int(r["lens"].sum())
        run = r["d_run"]
        e = [ev() for _ in range(4)] if marks is not None else None
        if e:
            e[0].record(stream)
        if separate_calls:
            c.step(r["d_ops"], n_ops, d_status, sid)
            c.translate(r["d_handles"], len(r["handles"]), d_pool, d_off, d_aoff, sid)
        else:       # the same two operations, the translation riding on the step's relocation-copy launch
            c.step_translate(r["d_ops"], n_ops, d_status, r["d_handles"], len(r["handles"]), d_pool, d_off, d_aoff, sid)
        if e:
            e[1].record(stream)
        if fused:
            c.gather_step(run, n_run, 0, m.n_attn_layers, out_k, out_v, kv_stride, cap_tok, d_cu,
                          0, m.n_ssm_layers, out_s, s_stride, out_c, c_stride, sid)
            if e:
                e[2].record(stream)
                e[3].record(stream)
                marks.append(e)
            return
        if per_layer:
            for l in range(m.n_attn_layers):
                c.gather_kv(l, run, n_run, out_k[l % lpl_kv], out_v[l % lpl_kv], cap_tok, d_cu, sid)
        else:
            for f, nl in kv_groups:
                c.gather_kv_layers(f, nl, run, n_run, out_k, out_v, kv_stride, cap_tok, d_cu, sid)
        if e:
            e[2].record(stream)
        if per_layer:
            for l in range(m.n_ssm_layers):
                c.gather_ssm(l, run, n_run, out_s[l % lpl_ssm], out_c[l % lpl_ssm], sid)
        else:
            for f, nl in ssm_groups:
                c.gather_ssm_layers(f, nl, run, n_run, out_s, s_stride, out_c, c_stride, sid)
        if e:
            e[3].record(stream)
            marks.append(e)

    def fresh_context(full_warmup=True):
        """A new context over the same arena, replayed up to the start of the timed window."""
        c = B.Context.from_workload(w, device=dev, arena=arena)
        for r in trace[:WS]:
            c.step(r["d_ops"], len(r["ops"]), d_status, sid)
        for r in trace[WS:WS + warmup]:
            if full_warmup:
                full_step(c, r, fused=one_launch)
            else:
                c.step(r["d_ops"], len(r["ops"]), d_status, sid)
        torch.cuda.synchronize(dev)
        return c

    timed = trace[WS + warmup:]

    # ---- timed region 1: K whole steps, one pair of events, nothing else on the stream ----
    ctx = fresh_context()
    reloc0 = ctx.stats()["relocated_bytes"]
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    torch.cuda.synchronize(dev)
    sampler = ClockSampler(dev.index or 0)
    sampler.start()
    launches0 = ctx.launch_count()
    e0, e1 = ev(), ev()
    e0.record(stream)
    for r in timed:
        full_step(ctx, r, fused=one_launch)
    e1.record(stream)
    torch.cuda.synchronize(dev)
    if world > 1:
        dist.barrier()
    total_ms = e0.elapsed_time(e1)
    launches = ctx.launch_count() - launches0
    st_b = ctx.stats()
    reloc_timed = st_b["relocated_bytes"] - reloc0
    ctx.close()

    # ---- region 2: the same window again with one event pair per kernel class and step ----
    def timed_classes(per_layer, fused=False):
        c = fresh_context()
        marks = []
        for r in timed:
            full_step(c, r, marks, per_layer=per_layer, fused=fused, separate_calls=per_layer)
        torch.cuda.synchronize(dev)
        st = c.stats()
        c.close()
        nl_kv = m.n_attn_layers if per_layer else len(kv_groups)
        nl_ssm = m.n_ssm_layers if per_layer else len(ssm_groups)
        return ({"step": [e[0].elapsed_time(e[1]) for e in marks],
                 "kv": [e[1].elapsed_time(e[2]) / nl_kv for e in marks],       # average per launch
                 "ssm": [e[2].elapsed_time(e[3]) / nl_ssm for e in marks]}, st)

    per, st_c = timed_classes(per_layer=False)
    per_l = timed_classes(per_layer=True)[0] if full else None
    per_f = timed_classes(per_layer=False, fused=True)[0] if one_launch else None

    # ---- region 3: the allocator part alone (avmp_step_translate per step, the calls back to back as a serving
    #      loop issues them; no events between steps, which would keep consecutive launches from overlapping) ----
    def alloc_only(separate):
        c = fresh_context(full_warmup=False)
        a0, a1 = ev(), ev()
        a0.record(stream)
        for r in timed:
            if separate:
                c.step(r["d_ops"], len(r["ops"]), d_status, sid)
                c.translate(r["d_handles"], len(r["handles"]), d_pool, d_off, d_aoff, sid)
            else:
                c.step_translate(r["d_ops"], len(r["ops"]), d_status, r["d_handles"], len(r["handles"]), d_pool, d_off, d_aoff, sid)
        a1.record(stream)
        torch.cuda.synchronize(dev)
        c.close()
        return a0.elapsed_time(a1)

    alloc_ms, alloc_sep_ms = alloc_only(False), alloc_only(True)
    clocks = sampler.stop()

    # ---- e2e: host buffers in, host results out, every step ----
    e2e_ms, h2d, d2h = None, 0, 0
    if full:
        ctx = fresh_context(full_warmup=False)
        pin = lambda a: torch.from_numpy(np.ascontiguousarray(a).view(np.uint8).reshape(-1).copy()).pin_memory()
        h_ops = [pin(r["ops"]) if len(r["ops"]) else torch.zeros(16, dtype=torch.uint8).pin_memory() for r in timed]
        h_run = [pin(r["run"]) if len(r["run"]) else torch.zeros(16, dtype=torch.uint8).pin_memory() for r in timed]
        h_status = torch.zeros(w.concurrency * 2 + 16, dtype=torch.int32).pin_memory()
        h_cu = torch.zeros(max_run + 1, dtype=torch.int32).pin_memory()
        d_run_buf = torch.zeros(max_run * 4 + 16, dtype=torch.uint8, device=dev)
        torch.cuda.synchronize(dev)
        t0 = time.perf_counter()
        for r, ho, hr in zip(timed, h_ops, h_run):
            n_ops, n_run = len(r["ops"]), len(r["run"])
            ctx.step_host(ho, n_ops, h_status, sid)                    # H2D ops, D2H statuses, sync
            d_run_buf[: n_run * 4].copy_(hr[: n_run * 4], non_blocking=True)   # H2D running list
            cap_tok = int(r["lens"].sum())
            if one_launch:
                ctx.gather_step(d_run_buf, n_run, 0, m.n_attn_layers, out_k, out_v, kv_stride, cap_tok, d_cu,
                                0, m.n_ssm_layers, out_s, s_stride, out_c, c_stride, sid)
            else:
                for f, nl in kv_groups:
                    ctx.gather_kv_layers(f, nl, d_run_buf, n_run, out_k, out_v, kv_stride, cap_tok, d_cu, sid)
                for f, nl in ssm_groups:
                    ctx.gather_ssm_layers(f, nl, d_run_buf, n_run, out_s, s_stride, out_c, c_stride, sid)
            h_cu[: n_run + 1].copy_(d_cu[: n_run + 1], non_blocking=True)   # D2H row offsets of the batch
            torch.cuda.synchronize(dev)
            h2d += n_ops * 12 + n_run * 4
            d2h += n_ops * 4 + (n_run + 1) * 4
        e2e_ms = (time.perf_counter() - t0) * 1e3
        ctx.close()

    # ---- accounting ----
    K = len(timed)
    by = [step_bytes(m, len(r["run"]), int(r["lens"].sum()), 0) for r in timed]
    kv_bytes = sum(b["kv"] for b in by)
    ssm_bytes = sum(b["ssm"] for b in by)
    res = {
        "K": K, "total_ms": total_ms, "e2e_ms": e2e_ms, "h2d": h2d, "d2h": d2h, "launches": launches,
        "kv_bytes": kv_bytes, "ssm_bytes": ssm_bytes, "reloc_bytes": reloc_timed,
        "moved": kv_bytes + ssm_bytes + 2 * reloc_timed,
        "n_ops": sum(len(r["ops"]) for r in timed), "units": sum(r["units"] for r in timed),
        "alloc_ms": alloc_ms, "alloc_sep_ms": alloc_sep_ms, "handles": sum(len(r["handles"]) for r in timed),
        "per": per, "per_l": per_l, "per_f": per_f, "one_launch": one_launch, "clocks": clocks, "lpl": (lpl_kv, lpl_ssm),
        "n_kv_launches": len(kv_groups), "n_ssm_launches": len(ssm_groups),
        "running_mean": float(np.mean([len(r["run"]) for r in timed])),
        "tokens_mean": float(np.mean([int(r["lens"].sum()) for r in timed])),
        "rebalances": st_c["n_rebalance"], "n_oom": st_c["n_oom"],
        "replay_matches": all(st_b[k] == stats_a[k] for k in stats_a if not k.startswith(("relocation_ns", "step_ns"))),
    }
    del out_k, out_v, out_s, out_c, arena, trace, timed
    torch.cuda.empty_cache()
    return res


def class_figures(res: dict, m: W.ModelShape, peak: float) -> dict:
    """GB/s and fractions of the copy-kernel classes of one measured workload, from bytes by definition of the
    operations and event-timed launch durations."""
    K = res["K"]
    per = res["per"]
    ssm_launch_bytes = res["ssm_bytes"] / (K * res["n_ssm_launches"])
    kv_launch_bytes = res["kv_bytes"] / (K * res["n_kv_launches"])
    ssm_ms, kv_ms, step_ms = float(np.mean(per["ssm"])), float(np.mean(per["kv"])), float(np.mean(per["step"]))
    out = {"ssm_gbs": ssm_launch_bytes / (ssm_ms * 1e-3) / 1e9, "ssm_launch_ms": ssm_ms, "ssm_launch_bytes": ssm_launch_bytes,
           "kv_gbs": kv_launch_bytes / (kv_ms * 1e-3) / 1e9, "kv_launch_ms": kv_ms, "kv_launch_bytes": kv_launch_bytes,
           "allocator_us_per_step": res["alloc_ms"] * 1e3 / K, "allocator_ops_per_s": res["n_ops"] / (res["alloc_ms"] * 1e-3),
           "allocator_us_per_step_separate_calls": res["alloc_sep_ms"] * 1e3 / K,
           "allocator_us_per_step_inside_full_steps": step_ms * 1e3,
           "unit_allocs_frees_per_s": res["units"] / (res["alloc_ms"] * 1e-3),
           "handles_translated_per_step": res["handles"] / K}
    if res["per_f"] is not None:
        ms = float(np.mean([a + b for a, b in zip(res["per_f"]["kv"], res["per_f"]["ssm"])]))   # kv mark is empty
        out["step_gather_gbs"] = (res["kv_bytes"] + res["ssm_bytes"]) / K / (ms * 1e-3) / 1e9
        out["step_gather_launch_ms"] = ms
    if res["per_l"] is not None:
        pl = res["per_l"]
        out["single_layer_ssm_gbs"] = (res["ssm_bytes"] / (K * m.n_ssm_layers)) / (float(np.mean(pl["ssm"])) * 1e-3) / 1e9
        out["single_layer_kv_gbs"] = (res["kv_bytes"] / (K * m.n_attn_layers)) / (float(np.mean(pl["kv"])) * 1e-3) / 1e9
        out["single_layer_ssm_launch_ms"] = float(np.mean(pl["ssm"]))
        out["single_layer_kv_launch_ms"] = float(np.mean(pl["kv"]))
    return out


def run_ours(args, rank: int, world: int, local_rank: int) -> dict:
    import torch
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    w = W.config(args.workload, seed=rank % 3 if world > 1 else args.seed)
    m = w.model
    peak, peak_kind = _peaks()
    res = measure(w, dev, steps=args.steps, warmup=args.warmup, warm_steps=args.warm_steps,
                  asked_lpl=args.layers_per_launch, full=True, world=world)
    K = res["K"]
    local_sums = np.array([res["moved"], res["n_ops"], res["kv_bytes"], res["ssm_bytes"], res["launches"],
                           res["h2d"], res["d2h"]], dtype=np.float64)
    total_ms_g, sums = reduce_over_ranks(res["total_ms"], local_sums, world)
    e2e_ms_g, _ = reduce_over_ranks(res["e2e_ms"], np.zeros(1), world)
    f = class_figures(res, m, peak)
    lpl_kv, lpl_ssm = res["lpl"]
    traffic = max(f["ssm_launch_bytes"] - L2_DIRTY_TAIL_BYTES, f["ssm_launch_bytes"] / 2)
    out = {
        "metric": METRIC, "value": sums[0] / (total_ms_g * 1e-3) / 1e9, "unit": "GB/s",
        "n_gpus": world, "steps": K, "warmup": args.warmup, "ms_per_step": total_ms_g / K,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u32",
        "data": "synthetic", "impl": "ours",
        "config": config_dict(w, args.warm_steps),
        "workload_stats": {"running_mean": res["running_mean"], "tokens_mean": res["tokens_mean"],
                           "ops_per_step": res["n_ops"] / K, "units_per_step": res["units"] / K,
                           "layers_per_launch": {"kv": lpl_kv, "ssm": lpl_ssm},
                           "relocated_bytes_in_window": int(res["reloc_bytes"]), "rebalances_total": res["rebalances"],
                           "n_oom_total": res["n_oom"], "replay_matches_closed_loop": res["replay_matches"]},
        "roofline": {"kernel": f"stream_bulk_kernel<SsmPieces<gather>> (avmp_gather_ssm_layers, {lpl_ssm} SSM layers per launch)",
                     "bound": "hbm", "achieved": f["ssm_gbs"], "peak": peak, "unit": "GB/s", "frac": f["ssm_gbs"] / peak,
                     "peak_source": f"MEASURED_PEAKS.json hbm_gbs ({peak_kind})",
                     "frac_of_nominal_8000": f["ssm_gbs"] / 8000.0, "avg_launch_ms": f["ssm_launch_ms"],
                     "bytes_per_launch": f["ssm_launch_bytes"], "traffic": traffic,
                     "traffic_source": "algorithmic bytes minus the ~47 MB of output still dirty in L2 at kernel end "
                                       "(ncu captures of this kernel at 1 GB and 6.8 GB per launch, profiles/); "
                                       "recorded from those captures, not measured in this run",
                     "secondary": {
                         "kv_gather": {"gbs": f["kv_gbs"], "frac": f["kv_gbs"] / peak, "avg_launch_ms": f["kv_launch_ms"],
                                       "bytes_per_launch": f["kv_launch_bytes"],
                                       "note": f"avmp_gather_kv_layers, {lpl_kv} attention layers per launch, plan computed inside the launch"},
                         "single_layer_ssm": {"gbs": f["single_layer_ssm_gbs"], "frac": f["single_layer_ssm_gbs"] / peak,
                                              "avg_launch_ms": f["single_layer_ssm_launch_ms"],
                                              "note": "same window, avmp_gather_ssm once per layer, back to back"},
                         "single_layer_kv": {"gbs": f["single_layer_kv_gbs"], "frac": f["single_layer_kv_gbs"] / peak,
                                             "avg_launch_ms": f["single_layer_kv_launch_ms"],
                                             "note": "same window, avmp_gather_kv once per layer, back to back"},
                         "step_gather": ({"gbs": f["step_gather_gbs"], "frac": f["step_gather_gbs"] / peak,
                                          "avg_launch_ms": f["step_gather_launch_ms"],
                                          "note": "avmp_gather_step: both gathers of all layers in one launch"}
                                         if "step_gather_gbs" in f else None),
                         "allocator_ops_per_s": f["allocator_ops_per_s"] * (world if world > 1 else 1),
                         "allocator_us_per_step": f["allocator_us_per_step"],
                         "allocator_us_per_step_separate_calls": f["allocator_us_per_step_separate_calls"],
                         "allocator_us_per_step_inside_full_steps": f["allocator_us_per_step_inside_full_steps"],
                         "handles_translated_per_step": f["handles_translated_per_step"],
                         "unit_allocs_frees_per_s": f["unit_allocs_frees_per_s"],
                         "allocator_note": "avmp_step_translate (allocator step + translate of every live handle of the batch; "
                                           "the translation rides on the step's relocation-copy launch), the window's steps "
                                           "issued back to back under one CUDA-event pair, rank 0's timing; separate_calls = "
                                           "avmp_step then avmp_translate; inside_full_steps = the same call between two events "
                                           "inside whole engine steps (the events keep it from overlapping its neighbours); units = KV pages + SSM blocks allocated "
                                           "or freed, counted from the request slots' net change per step"}},
        "e2e": {"value": sums[0] / (e2e_ms_g * 1e-3) / 1e9, "unit": "GB/s", "ms_per_step": e2e_ms_g / K,
                "h2d_bytes_per_step": sums[5] / K / world, "d2h_bytes_per_step": sums[6] / K / world,
                "note": "ops and running list from pinned host memory, statuses and row offsets back to the host every step; gathered batch buffers stay in HBM for the model's kernels"},
        "gpu_launches": int(sums[4]),
        "clocks": res["clocks"],
        "paper_context": "the paper (pure-Python prototype, one RTX 3060 12GB) reports 1.83-13.3x goodput and a 7.6 % "
                         "OOM reduction for dynamic rebalancing against its best static baseline; it reports no "
                         "allocator ops/s, GB/s or kernel timings, so vs_baseline is null",
    }
    return out


def other_configs(dev, skip: str) -> list:
    """The other configurations, each measured briefly the same way (K whole steps under one event pair, then
    per kernel class): whole-step GB/s and the fraction of the measured peak the two gathers reach."""
    peak, _ = _peaks()
    rows = []
    for name, (k, ws) in OTHER_CONFIGS.items():
        if name == skip:
            continue
        w = W.config(name)
        try:
            res = measure(w, dev, steps=k, warmup=3, warm_steps=ws, asked_lpl=0, full=False)
        except Exception as exc:      # a side measurement must not take the headline line down with it
            rows.append({"workload": name, "unavailable": f"{type(exc).__name__}: {exc}"})
            continue
        f = class_figures(res, w.model, peak)
        rows.append({"workload": name, "steps": res["K"], "timed_region_ms": res["total_ms"],
                     "value": res["moved"] / (res["total_ms"] * 1e-3) / 1e9, "frac": res["moved"] / (res["total_ms"] * 1e-3) / 1e9 / peak,
                     "ms_per_step": res["total_ms"] / res["K"],
                     "running_mean": res["running_mean"], "tokens_mean": res["tokens_mean"],
                     "ssm_gather_gbs": f["ssm_gbs"], "ssm_gather_frac": f["ssm_gbs"] / peak,
                     "kv_gather_gbs": f["kv_gbs"], "kv_gather_frac": f["kv_gbs"] / peak,
                     "step_gather_gbs": f.get("step_gather_gbs"),
                     "step_gather_frac": f["step_gather_gbs"] / peak if "step_gather_gbs" in f else None,
                     "gathers_per_step": "one launch (avmp_gather_step)" if res["one_launch"] else "one launch per kind and group of layers",
                     "allocator_us_per_step": f["allocator_us_per_step"], "allocator_ops_per_s": f["allocator_ops_per_s"],
                     "replay_matches_closed_loop": res["replay_matches"], "clocks": res["clocks"]})
    return rows


# ---------------------------------------------------------------------------------------
# micro-benchmarks reported beside the headline: one large migration, allocator rate vs batch
# ---------------------------------------------------------------------------------------
def migration_microbench(dev) -> dict:
    """Fill the KV store, free every other request so live pages are striped over the whole
    store, then exhaust the SSM store: one CapacityError cedes the top 16 384 KV pages and the
    migration must move every live page it finds there (about 2 GB)."""
    import torch
    from paper_2605_22416_b200 import binding as B
    m = W.JAMBA_LIKE
    ctx = B.Context(m, 16 * W.GiB, 0.3, 16384, max_requests=1024, max_pages=256, device=dev)
    s0 = ctx.stats()
    n_req = s0["cap_ssm"] // m.n_ssm_layers
    per = min(256, s0["cap_kv"] // n_req)
    st = np.zeros(1024, np.uint32)
    ctx.step_host(W.make_ops(W.OP_ADMIT, np.arange(n_req), per * 16), n_req, st)
    assert (st[:n_req] == 0).all()
    fin = np.arange(0, n_req, 2)
    ctx.step_host(W.make_ops(W.OP_FINISH, fin, 0), len(fin), st)
    ops = W.make_ops(W.OP_ADMIT, 512 + np.arange(n_req), 16)
    d_ops = torch.from_numpy(ops.view(np.uint8).reshape(-1)).to(dev)
    d_st = torch.zeros(n_req, dtype=torch.int32, device=dev)
    torch.cuda.synchronize(dev)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    ctx.step(d_ops, n_req, d_st)
    e1.record()
    torch.cuda.synchronize(dev)
    s = ctx.stats()
    ms = e0.elapsed_time(e1)
    ctx.close()
    moved = 2 * s["relocated_bytes"]
    peak, _ = _peaks()
    copy_s = s["relocation_ns_last"] * 1e-9
    return {"relocated_blocks": s["relocated_blocks"], "relocated_bytes": s["relocated_bytes"],
            "rebalances": s["n_rebalance"], "step_ms": ms,
            "gbs_whole_step": moved / (ms * 1e-3) / 1e9,
            "copy_kernel_ms_device_clock": copy_s * 1e3,
            "gbs_copy_kernel": moved / copy_s / 1e9 if copy_s > 0 else None,
            "frac_of_peak_copy_kernel": moved / copy_s / 1e9 / peak if copy_s > 0 else None,
            "note": "one avmp_step whose CapacityError migrates 16384 KV pages; whole step = plan kernel + copy "
                    "(CUDA events); copy kernel alone by the device clock stamped inside it (first warp in, last out)"}


def remap_microbench(dev, granules=(1, 2, 4, 8, 16, 32, 64), reps=7) -> dict:
    """What migrating capacity by remapping physical pages would cost on this machine (the paper's proposed
    alternative to oversized stores, Sections 3.2 / 4.6): two virtual ranges (the two stores), N physical
    granules unmapped from the donor's range and mapped into the recipient's with the CUDA virtual memory
    management calls, including the stream synchronisation the host needs before it may touch mappings the
    device might still be using (and to learn the device's decision at all).  Host wall clock, median of
    `reps`; 128 MiB of physical memory in total.  Compared by the caller with the relocation copy's time."""
    import torch
    from cuda.bindings import driver as cu

    def ck(r):
        err, rest = r[0], r[1:]
        if int(err) != 0:
            raise RuntimeError(f"CUDA driver call failed: {err}")
        return rest[0] if len(rest) == 1 else rest

    torch.cuda.synchronize(dev)
    prop = cu.CUmemAllocationProp()
    prop.type = cu.CUmemAllocationType.CU_MEM_ALLOCATION_TYPE_PINNED
    prop.location.type = cu.CUmemLocationType.CU_MEM_LOCATION_TYPE_DEVICE
    prop.location.id = dev.index or 0
    gran = int(ck(cu.cuMemGetAllocationGranularity(prop, cu.CUmemAllocationGranularity_flags.CU_MEM_ALLOC_GRANULARITY_MINIMUM)))
    n_max = max(granules)
    span = n_max * gran
    va = [int(ck(cu.cuMemAddressReserve(span, gran, 0, 0))) for _ in range(2)]     # donor range, recipient range
    handles = [ck(cu.cuMemCreate(gran, prop, 0)) for _ in range(n_max)]
    acc = cu.CUmemAccessDesc()
    acc.location.type = cu.CUmemLocationType.CU_MEM_LOCATION_TYPE_DEVICE
    acc.location.id = dev.index or 0
    acc.flags = cu.CUmemAccess_flags.CU_MEM_ACCESS_FLAGS_PROT_READWRITE
    where = 0                                       # which range the granules are mapped in
    flag = torch.zeros(2, dtype=torch.int64, device=dev)
    h_flag = torch.zeros(2, dtype=torch.int64).pin_memory()
    rows = []
    try:
        for i, h in enumerate(handles):
            ck(cu.cuMemMap(va[0] + i * gran, gran, 0, h, 0))
        ck(cu.cuMemSetAccess(va[0], span, [acc], 1))
        for n in granules:
            samples, sync_samples = [], []
            for _ in range(reps):
                src, dst = va[where], va[1 - where]
                torch.cuda.synchronize(dev)
                t0 = time.perf_counter()
                h_flag.copy_(flag, non_blocking=True)              # the device's decision reaches the host
                torch.cuda.synchronize(dev)
                t1 = time.perf_counter()
                for i in range(n):
                    ck(cu.cuMemUnmap(src + i * gran, gran))
                    ck(cu.cuMemMap(dst + i * gran, gran, 0, handles[i], 0))
                ck(cu.cuMemSetAccess(dst, n * gran, [acc], 1))
                t2 = time.perf_counter()
                samples.append((t2 - t0) * 1e6)
                sync_samples.append((t1 - t0) * 1e6)
                # back again (untimed), so that every sample starts from the same mapping
                for i in range(n):
                    ck(cu.cuMemUnmap(dst + i * gran, gran))
                    ck(cu.cuMemMap(src + i * gran, gran, 0, handles[i], 0))
                ck(cu.cuMemSetAccess(src, n * gran, [acc], 1))
            rows.append({"granules": n, "bytes": n * gran, "remap_us": float(np.median(samples)),
                         "of_which_sync_and_readback_us": float(np.median(sync_samples)),
                         "us_per_granule": (float(np.median(samples)) - float(np.median(sync_samples))) / n})
    finally:
        for i in range(n_max):                  # each granule is mapped in one of the two ranges (errors ignored)
            cu.cuMemUnmap(va[0] + i * gran, gran)
            cu.cuMemUnmap(va[1] + i * gran, gran)
        for h in handles:
            cu.cuMemRelease(h)
        for r in va:
            cu.cuMemAddressFree(r, span)
    return {"granule_bytes": gran, "rows": rows,
            "note": "host wall clock per migration of N granules: readback + stream sync, then cuMemUnmap + cuMemMap per "
                    "granule and one cuMemSetAccess for the range; no data moves"}


def relocation_small_cases(dev, batch_units=(8, 32, 128, 512, 2048)) -> list:
    """The copy path on the same byte counts: one migration of B KV pages (256 KiB each) out of a half-live
    store, timed as the whole avmp_step (plan kernel + copy, CUDA events) and as the copy kernel alone (device
    clock).  About half of the ceded pages are live and have to be copied."""
    import torch
    from paper_2605_22416_b200 import binding as B
    m = W.JAMBA_LIKE
    out = []
    for units in batch_units:
        ctx = B.Context(m, 4 * W.GiB, 0.3, units, max_requests=256, max_pages=256, device=dev)
        s0 = ctx.stats()
        n_req = s0["cap_ssm"] // m.n_ssm_layers
        per = min(256, s0["cap_kv"] // n_req)
        st = np.zeros(512, np.uint32)
        ctx.step_host(W.make_ops(W.OP_ADMIT, np.arange(n_req), per * 16), n_req, st)
        assert (st[:n_req] == 0).all()
        fin = np.arange(0, n_req, 2)
        ctx.step_host(W.make_ops(W.OP_FINISH, fin, 0), len(fin), st)
        ops = W.make_ops(W.OP_ADMIT, 128 + np.arange(n_req), 16)
        d_ops = torch.from_numpy(ops.view(np.uint8).reshape(-1)).to(dev)
        d_st = torch.zeros(n_req, dtype=torch.int32, device=dev)
        torch.cuda.synchronize(dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        ctx.step(d_ops, n_req, d_st)
        e1.record()
        torch.cuda.synchronize(dev)
        s = ctx.stats()
        ctx.close()
        out.append({"migration_batch_units": units, "ceded_bytes": s["migrated_bytes"], "relocated_bytes": s["relocated_bytes"],
                    "rebalances": s["n_rebalance"], "step_us": e0.elapsed_time(e1) * 1e3,
                    "copy_kernel_us_device_clock": s["relocation_ns_last"] / 1e3})
    return out


def device_closed_loop(dev, workload: str, steps: int = 3000) -> dict:
    """The whole serving loop on the device (batch built, allocator stepped and statuses folded back by
    kernels, no host round trip), dynamic rebalancing against the static partition on the same trace:
    requests completed in the same number of engine steps, and the device time those steps took."""
    import torch
    from paper_2605_22416_b200 import binding as B
    out = {"workload": workload, "steps": steps}
    for label, enabled in (("dynamic", True), ("static", False)):
        w = W.config(workload, migration_enabled=enabled)
        ctx = B.Context.from_workload(w, device=dev)
        if w.kind == "sessions":
            ses = W.make_sessions(w)
            dd = B.SessionDriver(ctx, ses.arrival_step, ses.n_turns, ses.turn_prompt, ses.turn_output,
                                 ses.turn_think, w.concurrency)
        else:
            reqs = W.make_requests(w, min(w.n_requests, 200_000))
            dd = B.DeviceDriver(ctx, reqs.prompt, reqs.output, w.concurrency)
        sid = torch.cuda.current_stream().cuda_stream
        torch.cuda.synchronize(dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            dd.step(sid)
        e1.record()
        torch.cuda.synchronize(dev)
        ms = e0.elapsed_time(e1)
        ds, st = dd.stats(), ctx.stats()
        # the same loop again, 100 steps captured once in a CUDA graph and replayed
        graph_us = None
        try:
            side = torch.cuda.Stream(device=dev)
            gr = torch.cuda.CUDAGraph()
            torch.cuda.synchronize(dev)
            with torch.cuda.stream(side):
                with torch.cuda.graph(gr, stream=side):
                    for _ in range(100):
                        dd.step(side)
                g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                g0.record(side)
                for _ in range(10):
                    gr.replay()
                g1.record(side)
            torch.cuda.synchronize(dev)
            graph_us = g0.elapsed_time(g1) * 1e3 / 1000
        except Exception as exc:          # graphs are an optimisation of the launch path, not part of the result
            graph_us = f"capture failed: {type(exc).__name__}"
        out[label] = {"completed": ds["completed"], "us_per_step_cuda_graph": graph_us, "n_oom": st["n_oom"], "rebalances": st["n_rebalance"],
                      "ops": st["op_counter"], "device_ms": ms, "us_per_step": ms * 1e3 / steps,
                      "ops_per_s": st["op_counter"] / (ms * 1e-3),
                      "completed_per_s_allocator_only": ds["completed"] / (ms * 1e-3),
                      "relocation_ms": st["relocation_ns_total"] / 1e6,
                      "allocator_kernel_ms": st["step_ns_total"] / 1e6,
                      "oom_retry_share_of_allocator_kernel": st["step_ns_oom_retry"] / max(st["step_ns_total"], 1),
                      "migration_plan_share_of_allocator_kernel": st["step_ns_migration_plan"] / max(st["step_ns_total"], 1)}
        dd.close()
        ctx.close()
    out["completed_ratio_dynamic_over_static"] = out["dynamic"]["completed"] / max(out["static"]["completed"], 1)
    out["note"] = ("allocator-only loop: no model kernels and no gathers run between steps, so the per-second figures "
                   "are a ceiling on scheduling rate, not serving goodput; the ratio of completed requests is the "
                   "event-deterministic part")
    return out


def write_side_microbench(dev) -> dict:
    """The write side and translate on their own: all-layer scatters of the same shapes the gathers
    move, and a million handle translations."""
    import torch
    from paper_2605_22416_b200 import binding as B
    m = W.JAMBA_LIKE
    ctx = B.Context(m, 8 * W.GiB, 0.6, 128, max_requests=256, max_pages=256, device=dev)
    n, tokens = 96, 2048
    st = np.zeros(n, np.uint32)
    ctx.step_host(W.make_ops(W.OP_ADMIT, np.arange(n), tokens), n, st)
    assert (st == 0).all()
    reqs = torch.arange(n, dtype=torch.int32, device=dev)
    tot = n * tokens
    kb = torch.empty((m.n_attn_layers, tot, m.kv_row_bytes), dtype=torch.uint8, device=dev)
    vb = torch.empty((m.n_attn_layers, tot, m.kv_row_bytes), dtype=torch.uint8, device=dev)
    sb = torch.empty((m.n_ssm_layers, n, m.state_bytes), dtype=torch.uint8, device=dev)
    cb = torch.empty((m.n_ssm_layers, n, m.conv_bytes), dtype=torch.uint8, device=dev)
    sid = torch.cuda.current_stream().cuda_stream
    peak, _ = _peaks()

    def timed(fn, reps=5):
        fn()
        torch.cuda.synchronize(dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize(dev)
        return e0.elapsed_time(e1) / reps

    kv_bytes = 2 * tot * 2 * m.kv_row_bytes * m.n_attn_layers
    ssm_bytes = 2 * n * (m.state_bytes + m.conv_bytes) * m.n_ssm_layers
    ms_kv = timed(lambda: ctx.scatter_kv_layers(0, m.n_attn_layers, reqs, None, n, kb, vb, tot * m.kv_row_bytes, sid))
    ms_ssm = timed(lambda: ctx.scatter_ssm_layers(0, m.n_ssm_layers, reqs, n, sb, n * m.state_bytes, cb,
                                                  n * m.conv_bytes, sid))
    # translate: every handle of the batch, repeated to a million entries
    t, _ = ctx.export_tables()
    chain = t["req_chain"].reshape(256, 256)
    handles = np.concatenate([chain[r, :t["req_npages"][r]] for r in range(n)] +
                             [t["req_ssm"].reshape(256, m.n_ssm_layers)[:n].reshape(-1)]).astype(np.uint32)
    handles = np.resize(handles, 1 << 20)
    d_h = torch.from_numpy(handles.view(np.int32)).to(dev)
    d_pool = torch.empty(len(handles), dtype=torch.int32, device=dev)
    d_off = torch.empty(len(handles), dtype=torch.int64, device=dev)
    d_aoff = torch.empty(len(handles), dtype=torch.int64, device=dev)
    ms_tr = timed(lambda: ctx.translate(d_h, len(handles), d_pool, d_off, d_aoff, sid))
    err = ctx.stats()["error_code"]
    ctx.close()
    return {"scatter_kv_layers_gbs": kv_bytes / (ms_kv * 1e-3) / 1e9, "scatter_kv_frac_of_peak": kv_bytes / (ms_kv * 1e-3) / 1e9 / peak,
            "scatter_ssm_layers_gbs": ssm_bytes / (ms_ssm * 1e-3) / 1e9, "scatter_ssm_frac_of_peak": ssm_bytes / (ms_ssm * 1e-3) / 1e9 / peak,
            "translate_handles_per_s": len(handles) / (ms_tr * 1e-3), "translate_us_per_million": ms_tr * 1e3,
            "device_error_code": err,
            "note": f"{n} requests x {tokens} tokens, all {m.n_attn_layers} attention / {m.n_ssm_layers} SSM layers per launch"}


def allocator_scaling(dev, batches=(32, 256, 1024, 4096), warm=120, timed=60) -> list:
    """avmp_step alone on closed-loop traces of growing step batch (small units so that
    thousands of requests fit): the path is latency-bound, so ops/s grows with the batch."""
    import torch
    from paper_2605_22416_b200 import binding as B
    out = []
    for n in batches:
        w = W.Workload(f"alloc_micro_{n}", W.SMALL_UNIT_MODEL, 1 * W.GiB, 0.5, 128, n, n, 24, "queue", 400 * n)
        ctx = B.Context.from_workload(w, device=dev)
        drv = W.ClosedLoopDriver(w)
        trace = []
        while not drv.done and drv.step < warm + timed:
            ops = drv.next_batch()
            st = np.zeros(len(ops), np.uint32)
            ctx.step_host(np.ascontiguousarray(ops), len(ops), st)
            drv.feed(st)
            trace.append(ops)
        s_a = ctx.stats()
        ctx.close()
        ctx = B.Context.from_workload(w, device=dev)
        d_ops = [torch.from_numpy(np.ascontiguousarray(o).view(np.uint8).reshape(-1)).to(dev) if len(o) else None for o in trace]
        d_st = torch.zeros(2 * n + 16, dtype=torch.int32, device=dev)
        sid = torch.cuda.current_stream().cuda_stream
        for o, d in zip(trace[:warm], d_ops[:warm]):
            ctx.step(d, len(o), d_st, sid)
        torch.cuda.synchronize(dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for o, d in zip(trace[warm:], d_ops[warm:]):
            ctx.step(d, len(o), d_st, sid)
        e1.record()
        torch.cuda.synchronize(dev)
        s_b = ctx.stats()
        ctx.close()
        n_ops = sum(len(o) for o in trace[warm:])
        ms = e0.elapsed_time(e1)
        out.append({"step_batch": n, "ops_per_step": n_ops / max(len(trace) - warm, 1), "us_per_step": ms * 1e3 / max(len(trace) - warm, 1),
                    "ops_per_s": n_ops / (ms * 1e-3), "n_oom": s_b["n_oom"], "rebalances": s_b["n_rebalance"],
                    "replay_matches": all(s_b[k] == s_a[k] for k in ("n_oom", "n_rebalance", "op_counter", "free_kv", "free_ssm"))})
    return out


# ---------------------------------------------------------------------------------------
# the oracle on the host cores: cpu_baseline leg and the --impl reference arm
# ---------------------------------------------------------------------------------------
def run_oracle(args, n_sample_steps: int, budget_s: float = 25.0, warmup_steps: int = 0,
               sample_bytes: float = 3.0e9) -> dict:
    """The oracle as it stands, single thread, on a bounded sample of the same workload: every sampled step
    runs the allocator update of the WHOLE batch, then translate and the all-layer gathers for the first
    requests of the running batch whose units fit in `sample_bytes` of host memory (the oracle keeps real
    stores; the whole batch of the large configurations would need more host memory than a box may have)."""
    from oracle.avmp_oracle import Oracle
    w = W.config(args.workload, seed=args.seed)
    m = w.model
    o = Oracle.from_workload(w, with_store=True)
    drv = W.ClosedLoopDriver(w, requests=W.make_requests(w, min(w.n_requests, 400 * w.concurrency))
                             if w.kind == "queue" else None)
    while not drv.done and drv.step < args.warm_steps:
        ops = drv.next_batch()
        drv.feed(o.step(ops))

    def sample_of(run, lens):
        per_req = m.n_ssm_layers * (m.state_bytes + m.conv_bytes) + lens * 2 * m.kv_row_bytes * m.n_attn_layers
        n = int(np.searchsorted(np.cumsum(per_req), sample_bytes, side="right"))
        return max(1, min(n, len(run)))

    # give every unit the sample can touch real bytes (the stores are committed lazily)
    run = drv.running_slots.astype(np.uint32)
    ns0 = sample_of(run, drv.len[run]) if len(run) else 0
    rng = np.random.default_rng(0)
    if ns0:
        srun, slens = run[:ns0], drv.len[run[:ns0]]
        kb = rng.integers(0, 256, (int(slens.sum()), m.kv_row_bytes), dtype=np.uint8)
        for l in range(m.n_attn_layers):
            o.scatter_kv(l, srun, np.zeros(ns0, np.uint32), kb, kb)
        sb = rng.integers(0, 256, (ns0, m.state_bytes), dtype=np.uint8)
        cb = rng.integers(0, 256, (ns0, m.conv_bytes), dtype=np.uint8)
        for l in range(m.n_ssm_layers):
            o.scatter_ssm(l, srun, sb, cb)
    moved = n_ops = 0
    t_alloc = t_total = 0.0
    steps = 0
    sampled, batch = [], []
    while steps < warmup_steps + n_sample_steps and t_total < budget_s and not drv.done:
        ops = drv.next_batch()
        t0 = time.perf_counter()
        st = o.step(ops)
        t1 = time.perf_counter()
        drv.feed(st)
        run = drv.running_slots.astype(np.uint32)
        if len(run) == 0:
            continue
        ns = sample_of(run, drv.len[run])
        run = run[:ns]
        lens = drv.len[run]
        tot = int(lens.sum())
        tb = o.tables()
        chain = tb["req_chain"].reshape(w.max_requests, w.max_pages)
        handles = np.concatenate([chain[r, :tb["req_npages"][r]] for r in run] +
                                 [tb["req_ssm"].reshape(w.max_requests, m.n_ssm_layers)[run].reshape(-1)])
        t3 = time.perf_counter()
        o.translate(handles)
        for l in range(m.n_attn_layers):
            o.gather_kv(l, run, tot)
        for l in range(m.n_ssm_layers):
            o.gather_ssm(l, run)
        t4 = time.perf_counter()
        steps += 1
        if steps <= warmup_steps:
            continue
        frac = ns / len(drv.running_slots)
        b = step_bytes(m, len(run), tot, 0)
        moved += b["kv"] + b["ssm"]
        n_ops += len(ops)
        t_alloc += t1 - t0
        t_total += (t1 - t0) * frac + (t4 - t3)          # the allocator's share for the sampled part of the batch
        sampled.append(ns)
        batch.append(len(drv.running_slots))
    k = max(steps - warmup_steps, 1)
    return {"value": moved / t_total / 1e9, "unit": "GB/s", "cores": 1, "host_cores": os.cpu_count(), "kind": "oracle",
            "sample": f"{k} consecutive engine steps of the same workload after {args.warm_steps} warm steps: allocator "
                      f"step of the whole batch, then translate + all-layer gathers for the first {int(np.mean(sampled or [0]))} of "
                      f"{int(np.mean(batch or [0]))} running requests (what fits in {sample_bytes / 1e9:.0f} GB of host stores); "
                      f"GB/s over the sampled requests' bytes, {t_total:.1f} s of CPU work",
            "allocator_ops_per_s": n_ops / t_alloc if t_alloc > 0 else None,
            "ms_per_step": t_total / k * 1e3, "steps": k}


def run_reference(args) -> dict:
    w = W.config(args.workload, seed=args.seed)
    base = run_oracle(args, n_sample_steps=args.steps, budget_s=240.0, warmup_steps=args.warmup)
    return {"metric": METRIC, "value": base["value"], "unit": "GB/s", "n_gpus": args.gpus, "steps": base["steps"],
            "warmup": args.warmup, "ms_per_step": base["ms_per_step"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "u32", "data": "synthetic", "impl": "reference",
            "config": config_dict(w, args.warm_steps),
            "cpu_baseline": {k: base[k] for k in ("value", "unit", "cores", "kind", "sample")},
            "roofline": {"secondary": {"allocator_ops_per_s": base["allocator_ops_per_s"]}},
            "note": "the CPU oracle as it stands, single thread; each step is a bounded sample of the workload's step",
            "e2e": {"value": base["value"], "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="scale")
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-micro", action="store_true", help="skip the micro-benchmarks and the other configurations")
    ap.add_argument("--layers-per-launch", type=int, default=0,
                    help="SSM / KV layers gathered per launch (0 = as many as fit beside the arena); "
                         "the batch buffers then hold that many layers and are reused by the next group")
    ap.add_argument("--warm-steps", type=int, default=WARM_STEPS, help="closed-loop steps before the timed window")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        if rank == 0:
            print(json.dumps(run_reference(args)), flush=True)
        return

    if world > 1:
        import torch
        import torch.distributed as dist
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    out = run_ours(args, rank, world, local_rank)
    if rank == 0:
        if not args.no_micro:
            import torch
            dev = torch.device("cuda", local_rank)
            sec = out["roofline"]["secondary"]
            for key, fn in (("relocation_copy", migration_microbench), ("allocator_vs_step_batch", allocator_scaling),
                            ("write_side", write_side_microbench)):
                try:
                    sec[key] = fn(dev)
                except Exception as exc:      # side measurements must not take the headline line down with them
                    sec[key] = {"unavailable": f"{type(exc).__name__}: {exc}"}
            try:
                sec["remap_vs_copy"] = {"remap": remap_microbench(dev), "copy": relocation_small_cases(dev)}
            except Exception as exc:          # the comparison is context for one design decision, not part of the path
                sec["remap_vs_copy"] = {"unavailable": f"{type(exc).__name__}: {exc}"}
            try:
                sec["closed_loop_device"] = device_closed_loop(dev, args.workload, 1500 if args.workload == "scale" else 3000)
            except Exception as exc:
                sec["closed_loop_device"] = {"unavailable": f"{type(exc).__name__}: {exc}"}
            out["roofline"]["other_configs"] = other_configs(dev, skip=args.workload)
        if not args.no_cpu_baseline:
            import torch
            torch.cuda.empty_cache()
            out["cpu_baseline"] = run_oracle(args, n_sample_steps=12)
        print(json.dumps(out), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

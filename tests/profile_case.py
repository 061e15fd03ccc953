"""Small, self-contained launches of each kernel for profiling (a few GB on the device,
a handful of launches): `python tests/profile_case.py <case>`.  Measurement tooling, not part of the library.

Cases: ssm_gather, kv_gather (one layer per launch), ssm_gather_fused, kv_gather_fused (several
layers per launch), step_gather (both kinds, all layers, one launch), relocate, step.  Every case builds a context through the
C ABI, brings it to a busy state with a few allocator steps and then launches the kernel
of interest `--repeat` times on different layers, so every launch reads cold data.
"""
from __future__ import annotations

import argparse

import numpy as np
import torch

import sys
from pathlib import Path

sys.path.insert(0, str(Path(__file__).resolve().parent.parent))

from paper_2605_22416_b200 import binding as B  # noqa: E402
from paper_2605_22416_b200 import workloads as W  # noqa: E402


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a).view(np.uint8).reshape(-1)).cuda()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("case", choices=["ssm_gather", "kv_gather", "ssm_gather_fused", "kv_gather_fused", "step_gather", "relocate", "step"])
    ap.add_argument("--repeat", type=int, default=6)
    ap.add_argument("--pool-gib", type=float, default=3.0)
    ap.add_argument("--layers", type=int, default=8, help="layers per launch in the fused cases")
    args = ap.parse_args()
    m = W.JAMBA_LIKE
    pool = int(args.pool_gib * W.GiB)
    ev = lambda: torch.cuda.Event(enable_timing=True)

    if args.case == "step_gather":
        # a small engine step: 40 requests x 600 tokens, every attention and SSM layer in ONE launch
        n_req, tokens = 40, 600
        ctx = B.Context(m, pool, 0.6, 128, max_requests=256, max_pages=256)
        s0 = ctx.stats()
        n_req = min(n_req, s0["cap_ssm"] // m.n_ssm_layers, s0["cap_kv"] // (tokens // 16 + 1))
        st = np.zeros(n_req, np.uint32)
        ctx.step_host(W.make_ops(W.OP_ADMIT, np.arange(n_req), tokens), n_req, st)
        assert (st == 0).all(), st
        reqs = _dev(np.random.default_rng(0).permutation(n_req).astype(np.uint32))
        tot = n_req * tokens
        cu = torch.zeros(n_req + 1, dtype=torch.int32, device="cuda")
        bufs = [(torch.empty((m.n_attn_layers, tot, m.kv_row_bytes), dtype=torch.uint8, device="cuda"),
                 torch.empty((m.n_attn_layers, tot, m.kv_row_bytes), dtype=torch.uint8, device="cuda"),
                 torch.empty((m.n_ssm_layers, n_req, m.state_bytes), dtype=torch.uint8, device="cuda"),
                 torch.empty((m.n_ssm_layers, n_req, m.conv_bytes), dtype=torch.uint8, device="cuda")) for _ in range(2)]
        nbytes = 2 * tot * 2 * m.kv_row_bytes * m.n_attn_layers + 2 * n_req * (m.state_bytes + m.conv_bytes) * m.n_ssm_layers
        for i in range(args.repeat):
            ok, ov, os_, oc = bufs[i % 2]
            a, b = ev(), ev()
            a.record()
            ctx.gather_step(reqs, n_req, 0, m.n_attn_layers, ok, ov, tot * m.kv_row_bytes, tot, cu,
                            0, m.n_ssm_layers, os_, n_req * m.state_bytes, oc, n_req * m.conv_bytes)
            b.record()
            torch.cuda.synchronize()
            print(f"step_gather launch {i}: {a.elapsed_time(b) * 1e3:.1f} us, {nbytes / 1e6:.0f} MB, "
                  f"{nbytes / a.elapsed_time(b) / 1e6:.0f} GB/s")
        print(ctx.stats())
        ctx.close()
        return

    if args.case in ("ssm_gather_fused", "kv_gather_fused"):
        kv = args.case == "kv_gather_fused"
        nl = min(args.layers, m.n_attn_layers if kv else m.n_ssm_layers)
        n_req, tokens = (48, 2048) if kv else (150, 64)
        ctx = B.Context(m, pool, 0.3 if kv else 0.85, 128, max_requests=256, max_pages=256)
        s0 = ctx.stats()
        n_req = min(n_req, s0["cap_ssm"] // m.n_ssm_layers, s0["cap_kv"] // (tokens // 16))
        st = np.zeros(n_req, np.uint32)
        ctx.step_host(W.make_ops(W.OP_ADMIT, np.arange(n_req), tokens), n_req, st)
        assert (st == 0).all(), st
        reqs = _dev(np.random.default_rng(0).permutation(n_req).astype(np.uint32))
        if kv:
            tot = n_req * tokens
            cu = torch.zeros(n_req + 1, dtype=torch.int32, device="cuda")
            ok = torch.empty((nl, tot, m.kv_row_bytes), dtype=torch.uint8, device="cuda")
            ov = torch.empty((nl, tot, m.kv_row_bytes), dtype=torch.uint8, device="cuda")
            nbytes = 2 * tot * 2 * m.kv_row_bytes * nl
        else:
            os_ = torch.empty((nl, n_req, m.state_bytes), dtype=torch.uint8, device="cuda")
            oc = torch.empty((nl, n_req, m.conv_bytes), dtype=torch.uint8, device="cuda")
            nbytes = 2 * n_req * (m.state_bytes + m.conv_bytes) * nl
        for i in range(args.repeat):
            first = (i * nl) % ((m.n_attn_layers if kv else m.n_ssm_layers) - nl + 1)
            a, b = ev(), ev()
            a.record()
            if kv:
                ctx.gather_kv_layers(first, nl, reqs, n_req, ok, ov, tot * m.kv_row_bytes, tot, cu)
            else:
                ctx.gather_ssm_layers(first, nl, reqs, n_req, os_, n_req * m.state_bytes, oc, n_req * m.conv_bytes)
            b.record()
            torch.cuda.synchronize()
            print(f"{args.case} launch {i} ({nl} layers from {first}): {a.elapsed_time(b) * 1e3:.1f} us, "
                  f"{nbytes / 1e6:.0f} MB, {nbytes / a.elapsed_time(b) / 1e6:.0f} GB/s")
        print(ctx.stats())
        ctx.close()
        return

    if args.case in ("ssm_gather", "kv_gather", "step"):
        split = 0.85 if args.case != "kv_gather" else 0.3
        n_req = 150 if args.case != "kv_gather" else 48
        tokens = 64 if args.case != "kv_gather" else 2048
        ctx = B.Context(m, pool, split, 128, max_requests=256, max_pages=256)
        s0 = ctx.stats()
        n_req = min(n_req, s0["cap_ssm"] // m.n_ssm_layers, s0["cap_kv"] // (tokens // 16))
        ops = W.make_ops(W.OP_ADMIT, np.arange(n_req), tokens)
        st = np.zeros(n_req, np.uint32)
        ctx.step_host(ops, n_req, st)
        assert (st == 0).all(), st
        reqs = _dev(np.arange(n_req, dtype=np.uint32))
        if args.case == "ssm_gather":
            outs = [(torch.empty((n_req, m.state_bytes), dtype=torch.uint8, device="cuda"),
                     torch.empty((n_req, m.conv_bytes), dtype=torch.uint8, device="cuda")) for _ in range(args.repeat)]
            nbytes = 2 * n_req * (m.state_bytes + m.conv_bytes)
            for i in range(args.repeat):
                a, b = ev(), ev()
                a.record()
                ctx.gather_ssm(i % m.n_ssm_layers, reqs, n_req, outs[i][0], outs[i][1])
                b.record()
                torch.cuda.synchronize()
                print(f"ssm_gather launch {i}: {a.elapsed_time(b) * 1e3:.1f} us, {nbytes / a.elapsed_time(b) / 1e6:.0f} GB/s")
        elif args.case == "kv_gather":
            tot = n_req * tokens
            cu = torch.zeros(n_req + 1, dtype=torch.int32, device="cuda")
            outs = [(torch.empty((tot, m.kv_row_bytes), dtype=torch.uint8, device="cuda"),
                     torch.empty((tot, m.kv_row_bytes), dtype=torch.uint8, device="cuda")) for _ in range(min(args.repeat, 4))]
            nbytes = 2 * tot * 2 * m.kv_row_bytes
            for i in range(len(outs)):
                a, b = ev(), ev()
                a.record()
                ctx.gather_kv(i % m.n_attn_layers, reqs, n_req, outs[i][0], outs[i][1], tot, cu)
                b.record()
                torch.cuda.synchronize()
                print(f"kv_gather launch {i}: {a.elapsed_time(b) * 1e3:.1f} us, {nbytes / a.elapsed_time(b) / 1e6:.0f} GB/s")
        else:
            d_st = torch.zeros(n_req, dtype=torch.int32, device="cuda")
            ext = _dev(W.make_ops(W.OP_EXTEND, np.arange(n_req), 1))
            for i in range(args.repeat):
                a, b = ev(), ev()
                a.record()
                ctx.step(ext, n_req, d_st)
                b.record()
                torch.cuda.synchronize()
                print(f"step launch {i}: {a.elapsed_time(b) * 1e3:.1f} us for {n_req} ops")
        print(ctx.stats())
        ctx.close()
        return

    # relocate: fill the KV store, free every other long request so live pages are spread over
    # the whole store, then exhaust the SSM store: the migration cedes the top of the KV store
    # and must move the live pages it finds there.
    B_units = 4096
    ctx = B.Context(m, pool, 0.3, B_units, max_requests=512, max_pages=256)
    s0 = ctx.stats()
    n_req = min(400, s0["cap_ssm"] // m.n_ssm_layers)
    per = min(256, s0["cap_kv"] // n_req)
    st = np.zeros(512, np.uint32)
    ctx.step_host(W.make_ops(W.OP_ADMIT, np.arange(n_req), per * 16), n_req, st)
    assert (st[:n_req] == 0).all(), st[:n_req]
    ctx.step_host(W.make_ops(W.OP_FINISH, np.arange(0, n_req, 2), 0), (n_req + 1) // 2, st)
    n_new = n_req                      # more admits than the SSM store can hold: forces KV -> SSM
    d_ops = _dev(W.make_ops(W.OP_ADMIT, 256 + np.arange(n_new), 16))
    d_st = torch.zeros(n_new, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    a, b = ev(), ev()
    a.record()
    ctx.step(d_ops, n_new, d_st)
    b.record()
    torch.cuda.synchronize()
    s = ctx.stats()
    ms = a.elapsed_time(b)
    print(f"step with migration: {ms * 1e3:.1f} us; relocated {s['relocated_blocks']} blocks, "
          f"{s['relocated_bytes'] / 1e6:.1f} MB; rebalances {s['n_rebalance']}; "
          f">= {2 * s['relocated_bytes'] / ms / 1e6:.0f} GB/s (whole step time as the denominator)")
    ctx.close()


if __name__ == "__main__":
    main()

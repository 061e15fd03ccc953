"""The C ABI driven by a program that uses only the CUDA runtime (no PyTorch, no Python): it is
compiled with nvcc, run, and everything it prints -- per-op statuses, row offsets, counters, hashes of
the bytes it gathered after a migration had relocated them -- is compared with the oracle fed the same
operations and the same byte pattern."""
from __future__ import annotations

import os
import shutil
import subprocess
from pathlib import Path

import numpy as np
import pytest

from oracle.avmp_oracle import Oracle
from paper_2605_22416_b200 import workloads as W

ROOT = Path(__file__).resolve().parent.parent


def _fnv(a: np.ndarray) -> int:
    h = 1469598103934665603
    for b in a.reshape(-1).tolist():
        h = ((h ^ b) * 1099511628211) & 0xFFFFFFFFFFFFFFFF
    return h


def _ops(lst):
    a = np.zeros(len(lst), W.OP_DTYPE)
    for i, (k, f, r, t) in enumerate(lst):
        a[i] = (k, f, 0, r, t)
    return a


@pytest.mark.gpu
def test_plain_cuda_caller_matches_the_oracle():
    from paper_2605_22416_b200 import build
    lib = build.build_library()
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    exe = Path(os.environ.get("TMPDIR", "/tmp")) / f"avmp_plain_cuda_caller_{os.getpid()}"
    subprocess.check_call([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-std=c++17", f"-I{ROOT / 'include'}",
                           str(ROOT / "tests" / "plain_cuda_caller.cu"), "-o", str(exe), str(lib),
                           "-Xlinker", f"-rpath={lib.parent}"])
    out = subprocess.check_output([str(exe)], timeout=120).decode()
    exe.unlink()
    got = {}
    for line in out.splitlines():
        for kv in line.split():
            k, _, v = kv.partition("=")
            got[k] = v
    assert got.get("done") == "1", out

    # the same run on the oracle
    m = W.PR1_MODEL
    o = Oracle(m, 24 * W.MiB, 0.5, 6, max_requests=16, max_pages=48, min_rebalance_interval_ops=4, with_store=True)
    A, E, F = W.OP_ADMIT, W.OP_EXTEND, W.OP_FINISH
    st = []
    st += o.step(_ops([(A, 0, 0, 736), (A, 0, 1, 16)])).tolist()
    st += o.step(_ops([(F, 0, 0, 0), (A, 0, 2, 16), (A, 0, 3, 20), (A, 0, 4, 5), (A, 0, 5, 16), (A, 0, 6, 16),
                       (E, 0, 9, 5), (A, 0, 6, 1)])).tolist()
    reqs, lens = np.array([3, 1, 2], np.uint32), [20, 16, 16]
    row = m.kv_row_bytes
    k = np.concatenate([((r * 131 + np.arange(l)[:, None] * 7 + np.arange(row)[None, :]) & 255).astype(np.uint8)
                        for r, l in zip(reqs.tolist(), lens)])
    v = k ^ 0x5A
    state = np.stack([((r * 17 + np.arange(m.state_bytes) * 3) & 255).astype(np.uint8) for r in reqs.tolist()])
    conv = np.stack([(~(r * 17 + np.arange(m.conv_bytes) * 3) & 255).astype(np.uint8) for r in reqs.tolist()])
    assert o.scatter_kv(1, reqs, np.zeros(3, np.uint32), k, v) == 0
    assert o.scatter_ssm(2, reqs, state, conv) == 0
    last = o.step(_ops([(A, 0, 7, 30), (E, 0, 4, 100), (A, 0, 8, 16), (F, W.FLAG_KEEP_KV, 5, 0),
                        (A, W.FLAG_RESUME, 5, 40)])).tolist()
    s = o.stats()
    assert s["n_rebalance"] == 1 and s["relocated_blocks"] == 5       # the scenario does what its comments say
    ok, ov, ocu, bad = o.gather_kv(1, reqs, sum(lens))
    os_, oc, bad2 = o.gather_ssm(2, reqs)
    assert bad == 0 and bad2 == 0 and np.array_equal(ok, k) and np.array_equal(os_, state)

    assert got["statuses"] == "".join(f"{x}," for x in st)
    assert got["last_statuses"] == "".join(f"{x}," for x in last)
    assert got["cu"] == "".join(f"{x}," for x in ocu.tolist())
    assert (got["k_equal"], got["v_equal"], got["state_equal"], got["conv_equal"]) == ("1", "1", "1", "1")
    assert int(got["hash_k"]) == _fnv(ok) and int(got["hash_v"]) == _fnv(ov)
    assert int(got["hash_state"]) == _fnv(os_) and int(got["hash_conv"]) == _fnv(oc)
    for key, name in (("op_counter", "op_counter"), ("n_oom", "n_oom"), ("n_rebalance", "n_rebalance"),
                      ("relocated_blocks", "relocated_blocks"), ("cap_kv", "cap_kv"), ("cap_ssm", "cap_ssm"),
                      ("free_kv", "free_kv"), ("free_ssm", "free_ssm"), ("gap", "gap_bytes"), ("error_code", None)):
        assert int(got[key]) == (0 if name is None else s[name]), key

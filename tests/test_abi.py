"""Host-side checks that need no GPU: the C-ABI library builds, loads and exports every
symbol the public header declares; the layout arithmetic agrees with the closed forms; the
benchmark's cross-rank reduction works over a 2-rank gloo group."""
from __future__ import annotations

import ctypes
import os
import re
import subprocess
import sys
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent
GOLDEN = ROOT / "tests" / "golden"


def _lib():
    from paper_2605_22416_b200 import build
    return ctypes.CDLL(str(build.build_library()))


def test_library_exports_every_declared_symbol():
    header = (ROOT / "include" / "avmp.h").read_text()
    declared = re.findall(r"AVMP_API\s+[\w\s\*]+?\b(avmp_\w+)\s*\(", header)
    assert len(declared) >= 19 and "avmp_step" in declared and "avmp_gather_kv" in declared
    lib = _lib()
    for name in declared:
        assert hasattr(lib, name), f"{name} is declared in avmp.h but not exported"


def test_public_header_is_plain_c():
    """The boundary is a C ABI: avmp.h must compile as C99 (and as C++) on its own."""
    hdr = str(ROOT / "include" / "avmp.h")
    subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror", "-fsyntax-only", "-x", "c", hdr])
    subprocess.check_call(["g++", "-std=c++14", "-Wall", "-Werror", "-fsyntax-only", "-x", "c++", hdr])
    # and a C program can link against the library without any CUDA header
    src = ROOT / "tests" / "c_abi_smoke.c"
    from paper_2605_22416_b200 import build
    lib = build.build_library()
    exe = Path(os.environ.get("TMPDIR", "/tmp")) / f"avmp_c_abi_smoke_{os.getpid()}"
    subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Werror", f"-I{ROOT / 'include'}", str(src), "-o", str(exe),
                           str(lib), f"-Wl,-rpath,{lib.parent}"])
    out = subprocess.check_output([str(exe)]).decode()
    exe.unlink()
    assert "U_kv=262144 U_ssm=622592 kv_cap=8192 ssm_cap=3449" in out and "workspace_bytes=" in out
    # the ctypes declarations of the binding have the sizes the C compiler gives the header's structs
    # (the binding module needs no GPU to import; only its structure classes are used here)
    from paper_2605_22416_b200 import binding as B
    sizes = dict(kv.split("=") for kv in re.search(r"sizeof (.*)", out).group(1).split())
    from paper_2605_22416_b200 import workloads as W
    for name, n in sizes.items():
        mine = W.OP_DTYPE.itemsize if name == "avmp_op" else ctypes.sizeof(getattr(B, name))   # ops travel as a numpy record
        assert mine == int(n), (name, n, mine)


def test_binding_declares_every_symbol():
    src = (ROOT / "paper_2605_22416_b200" / "binding.py").read_text()
    header = (ROOT / "include" / "avmp.h").read_text()
    for name in re.findall(r"AVMP_API\s+[\w\s\*]+?\b(avmp_\w+)\s*\(", header):
        assert f'"{name}"' in src, f"binding.py does not bind {name}"


def test_layout_arithmetic_matches_closed_forms():
    """avmp_derive_layout is host arithmetic: check it against the hand-worked table."""
    from paper_2605_22416_b200 import workloads as W

    class Spec(ctypes.Structure):
        _fields_ = [(n, ctypes.c_uint32) for n in (
            "n_attn_layers", "n_ssm_layers", "page_tokens", "kv_heads", "head_dim", "kv_elem_bytes",
            "ssm_state_elems", "ssm_conv_elems", "ssm_elem_bytes")]

    class Layout(ctypes.Structure):
        _fields_ = [("pool_bytes_aligned", ctypes.c_uint64), ("unit_bytes", ctypes.c_uint64 * 2),
                    ("vid_space", ctypes.c_uint64 * 2), ("cap0", ctypes.c_uint64 * 2), ("gap0", ctypes.c_uint64),
                    ("kv_layer_bytes", ctypes.c_uint64), ("kv_row_bytes", ctypes.c_uint64),
                    ("ssm_state_bytes", ctypes.c_uint64), ("ssm_conv_bytes", ctypes.c_uint64)]

    lib = _lib()
    lib.avmp_derive_layout.argtypes = [ctypes.POINTER(Spec), ctypes.c_uint64, ctypes.c_double, ctypes.POINTER(Layout)]
    for line in (GOLDEN / "config_sizes.txt").read_text().splitlines():
        if not line.strip() or line.startswith("#"):
            continue
        name, u_kv, u_ssm, split, kv_cap, ssm_cap, v_kv, v_ssm = line.split()
        w = W.config(name)
        spec = Spec(*(getattr(w.model, f[0]) for f in Spec._fields_))
        out = Layout()
        assert lib.avmp_derive_layout(ctypes.byref(spec), w.pool_bytes, float(split), ctypes.byref(out)) == 0
        assert list(out.unit_bytes) == [int(u_kv), int(u_ssm)]
        assert list(out.cap0) == [int(kv_cap), int(ssm_cap)]
        assert list(out.vid_space) == [int(v_kv), int(v_ssm)]
        assert out.cap0[0] * out.unit_bytes[0] + out.cap0[1] * out.unit_bytes[1] + out.gap0 == out.pool_bytes_aligned
    # misuse the host can see
    out = Layout()
    spec = Spec(1, 1, 16, 1, 1, 2, 20, 4, 4)
    assert lib.avmp_derive_layout(ctypes.byref(spec), 1024, 1.5, ctypes.byref(out)) == -1
    assert lib.avmp_derive_layout(ctypes.byref(spec), 32, 0.5, ctypes.byref(out)) == -1
    lib.avmp_error_string.restype = ctypes.c_char_p
    assert lib.avmp_error_string(-2) == b"workspace too small"


_RANK_SCRIPT = r"""
import os, sys
sys.path.insert(0, {root!r})
import numpy as np
import torch.distributed as dist
import bench
dist.init_process_group("gloo", rank=int(os.environ["RANK"]), world_size=2)
r = dist.get_rank()
ms, sums = bench.reduce_over_ranks(10.0 + 5.0 * r, np.array([100.0 * (r + 1), 7.0]), 2)
assert ms == 15.0 and sums.tolist() == [300.0, 14.0], (ms, sums)
dist.barrier()
dist.destroy_process_group()
print("rank", r, "ok")
"""


def test_replica_reduction_over_two_gloo_ranks(tmp_path):
    """Multi-GPU is replicas only: the benchmark sums the work of all ranks and takes the
    slowest rank's time.  Two CPU ranks over gloo exercise exactly that reduction."""
    script = tmp_path / "rank.py"
    script.write_text(_RANK_SCRIPT.format(root=str(ROOT)))
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29731", WORLD_SIZE="2")
    procs = [subprocess.Popen([sys.executable, str(script)], env=dict(env, RANK=str(r)),
                              stdout=subprocess.PIPE, stderr=subprocess.STDOUT) for r in range(2)]
    outs = [p.communicate(timeout=120)[0].decode() for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    assert all("ok" in o for o in outs)


def test_plain_cuda_caller_compiles_and_links():
    """The CUDA-runtime-only caller of the ABI builds against the header and the library here (no GPU
    needed to compile; the GPU test runs it)."""
    import shutil
    from paper_2605_22416_b200 import build
    lib = build.build_library()
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    exe = Path(os.environ.get("TMPDIR", "/tmp")) / f"avmp_plain_cuda_caller_build_{os.getpid()}"
    subprocess.check_call([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-std=c++17", f"-I{ROOT / 'include'}",
                           str(ROOT / "tests" / "plain_cuda_caller.cu"), "-o", str(exe), str(lib),
                           "-Xlinker", f"-rpath={lib.parent}"])
    assert exe.exists()
    exe.unlink()

"""The gather entry point that keeps its scratch inside the library (for callers that
cannot allocate device memory or lend any): its output must equal the regular entry
point's, byte for byte, on two calls in a row that share the same in-library scratch.

Collected last on purpose: if it fails, a run that stops at the first failure has
already run every other test.  It builds its own context, so it passes alone in a
fresh process as well as after the rest of the suite."""
from __future__ import annotations

import numpy as np
import pytest

from paper_2605_22416_b200 import workloads as W

pytestmark = pytest.mark.gpu


def test_static_scratch_gather_matches_regular_gather_twice():
    import torch
    from paper_2605_22416_b200 import binding as B

    assert torch.cuda.is_available()
    dev = torch.device("cuda:0")
    m = W.PR1_MODEL
    ctx = B.Context(m, 96 * W.MiB, 0.5, 8, max_requests=64, max_pages=40, device=dev)
    # ragged lengths: partial last pages, one-token requests, exact page multiples
    lens = np.array([1, 15, 16, 17, 33, 100, 250, 512, 31, 64, 5, 199], np.uint32)
    n = len(lens)
    st = np.zeros(n, np.uint32)
    ctx.step_host(W.make_ops(W.OP_ADMIT, np.arange(n), lens), n, st)
    assert (st == 0).all()
    # finish a few and admit again so chains are not in slot order any more
    ctx.step_host(W.make_ops(W.OP_FINISH, [1, 4, 7], 0), 3, st)
    lens[[1, 4, 7]] = [77, 300, 9]
    ctx.step_host(W.make_ops(W.OP_ADMIT, [7, 1, 4], lens[[7, 1, 4]]), 3, st)
    assert (st[:3] == 0).all()
    rng = np.random.default_rng(11)
    tot = int(lens.sum())
    all_reqs = torch.arange(n, dtype=torch.int32, device=dev)
    for layer in range(m.n_attn_layers):
        kb = torch.from_numpy(rng.integers(0, 256, (tot, m.kv_row_bytes), dtype=np.uint8)).to(dev)
        vb = torch.from_numpy(rng.integers(0, 256, (tot, m.kv_row_bytes), dtype=np.uint8)).to(dev)
        ctx.scatter_kv(layer, all_reqs, None, n, kb, vb)

    def both(layer, req_ids, cap):
        reqs = torch.tensor(req_ids, dtype=torch.int32, device=dev)
        outs = []
        for fn in (ctx.gather_kv, ctx.gather_kv_static):
            k = torch.full((max(cap, 1), m.kv_row_bytes), 0xAB, dtype=torch.uint8, device=dev)
            v = torch.full((max(cap, 1), m.kv_row_bytes), 0xCD, dtype=torch.uint8, device=dev)
            cu = torch.full((len(req_ids) + 1,), -1, dtype=torch.int32, device=dev)
            fn(layer, reqs, len(req_ids), k, v, cap, cu)
            torch.cuda.synchronize()
            outs.append((k.cpu().numpy(), v.cpu().numpy(), cu.cpu().numpy()))
        (k0, v0, c0), (k1, v1, c1) = outs
        assert np.array_equal(c0, c1)
        assert np.array_equal(k0, k1) and np.array_equal(v0, v1)
        return c0

    # first call: the whole batch; second call right after it: a shorter, reordered list on
    # another layer, so anything left over in the shared scratch would show
    cu = both(0, list(range(n)), tot)
    assert cu[-1] == tot
    cu2 = both(3, [7, 0, 11, 3], int(lens[[7, 0, 11, 3]].sum()))
    assert cu2.tolist() == np.concatenate([[0], np.cumsum(lens[[7, 0, 11, 3]])]).tolist()
    # error items behave alike: an empty slot in the list, and a buffer that is too small
    e0 = ctx.stats()["error_count"]
    both(1, [0, 40, 2], int(lens[[0, 2]].sum()))
    both(2, [5, 6], int(lens[5]))
    assert ctx.stats()["error_count"] - e0 == 4      # one per bad item, from each entry point
    # a list beyond the fixed scratch is refused and nothing runs
    big = torch.zeros(B.AVMP_STATIC_GATHER_MAX_REQS + 1, dtype=torch.int32, device=dev)
    with pytest.raises(B.AvmpError, match="fixed in-library scratch"):
        ctx.gather_kv_static(0, big, B.AVMP_STATIC_GATHER_MAX_REQS + 1, big, big, 0, big)
    ctx.close()

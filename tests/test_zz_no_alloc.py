"""The gather entry point that keeps its scratch inside the library (for callers that
cannot allocate device memory or lend any): its output must equal the regular entry
point's and the CPU oracle's, byte for byte, on calls in a row that share the same
in-library scratch.

Collected last on purpose: if it fails, a run that stops at the first failure has
already run every other test.  It builds its own contexts, so it passes alone in a
fresh process as well as after the rest of the suite."""
from __future__ import annotations

import numpy as np
import pytest

from paper_2605_22416_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _three_way(ctx, o, m, dev, layer, req_ids, cap):
    """The regular entry point, the static-scratch entry point and the oracle on one request list:
    row offsets, K and V bytes (rows nobody wrote keep the fill pattern) and the number of error items."""
    import torch
    reqs = torch.tensor(np.asarray(req_ids, np.int64), dtype=torch.int32, device=dev)
    n = len(req_ids)
    outs, errs = [], []
    for fn in (ctx.gather_kv, ctx.gather_kv_static):
        k = torch.full((max(cap, 1), m.kv_row_bytes), 0xAB, dtype=torch.uint8, device=dev)
        v = torch.full((max(cap, 1), m.kv_row_bytes), 0xCD, dtype=torch.uint8, device=dev)
        cu = torch.full((n + 1,), -1, dtype=torch.int32, device=dev)
        e0 = ctx.stats()["error_count"]
        fn(layer, reqs, n, k, v, cap, cu)
        torch.cuda.synchronize()
        errs.append(ctx.stats()["error_count"] - e0)
        outs.append((k.cpu().numpy()[:cap], v.cpu().numpy()[:cap], cu.cpu().numpy().view(np.uint32)))
    (k0, v0, c0), (k1, v1, c1) = outs
    assert np.array_equal(c0, c1) and np.array_equal(k0, k1) and np.array_equal(v0, v1)
    assert errs[0] == errs[1]
    ok, ov, ocu, obad = o.gather_kv(layer, np.asarray(req_ids, np.uint32), cap)
    assert np.array_equal(c1, ocu) and errs[1] == obad
    # the oracle's buffers start as zeros, the device buffers as a fill pattern: compare the rows of the
    # requests that were copied (a request that does not fit, or holds nothing, copies nothing anywhere)
    for i in range(n):
        a, b = int(ocu[i]), int(ocu[i + 1])
        if b <= cap and b > a:
            assert np.array_equal(k1[a:b], ok[a:b]) and np.array_equal(v1[a:b], ov[a:b]), f"request {i} of the list"
    return c1


def test_static_scratch_gather_matches_regular_gather_and_oracle():
    import torch
    from oracle.avmp_oracle import Oracle
    from paper_2605_22416_b200 import binding as B

    assert torch.cuda.is_available()
    dev = torch.device("cuda:0")
    m = W.PR1_MODEL
    kw = dict(max_requests=64, max_pages=40)
    ctx = B.Context(m, 96 * W.MiB, 0.5, 8, device=dev, **kw)
    o = Oracle(m, 96 * W.MiB, 0.5, 8, with_store=True, **kw)
    # ragged lengths: partial last pages, one-token requests, exact page multiples
    lens = np.array([1, 15, 16, 17, 33, 100, 250, 512, 31, 64, 5, 199], np.uint32)
    n = len(lens)
    st = np.zeros(n, np.uint32)

    def both_step(ops):
        ctx.step_host(ops, len(ops), st)
        assert np.array_equal(st[:len(ops)], o.step(ops)) and (st[:len(ops)] == 0).all()

    both_step(W.make_ops(W.OP_ADMIT, np.arange(n), lens))
    # finish a few and admit again so chains are not in slot order any more
    both_step(W.make_ops(W.OP_FINISH, [1, 4, 7], 0))
    lens[[1, 4, 7]] = [77, 300, 9]
    both_step(W.make_ops(W.OP_ADMIT, [7, 1, 4], lens[[7, 1, 4]]))
    rng = np.random.default_rng(11)
    tot = int(lens.sum())
    all_reqs = torch.arange(n, dtype=torch.int32, device=dev)
    for layer in range(m.n_attn_layers):
        kb = rng.integers(0, 256, (tot, m.kv_row_bytes), dtype=np.uint8)
        vb = rng.integers(0, 256, (tot, m.kv_row_bytes), dtype=np.uint8)
        ctx.scatter_kv(layer, all_reqs, None, n, torch.from_numpy(kb).to(dev), torch.from_numpy(vb).to(dev))
        assert o.scatter_kv(layer, np.arange(n), np.zeros(n, np.uint32), kb, vb) == 0

    # first call: the whole batch; second call right after it: a shorter, reordered list on
    # another layer, so anything left over in the shared scratch would show
    cu = _three_way(ctx, o, m, dev, 0, list(range(n)), tot)
    assert cu[-1] == tot
    cu2 = _three_way(ctx, o, m, dev, 3, [7, 0, 11, 3], int(lens[[7, 0, 11, 3]].sum()))
    assert cu2.tolist() == np.concatenate([[0], np.cumsum(lens[[7, 0, 11, 3]])]).tolist()
    # error items behave alike: an empty slot in the list, and a buffer that is too small
    e0 = ctx.stats()["error_count"]
    _three_way(ctx, o, m, dev, 1, [0, 40, 2], int(lens[[0, 2]].sum()))
    _three_way(ctx, o, m, dev, 2, [5, 6], int(lens[5]))
    assert ctx.stats()["error_count"] - e0 == 4      # one per bad item, from each entry point
    # an empty list: only cu_seqlens[0] is written
    assert _three_way(ctx, o, m, dev, 0, [], 0).tolist() == [0]
    # a list beyond the fixed scratch is refused and nothing runs; so is one longer than the slot table
    big = torch.zeros(B.AVMP_STATIC_GATHER_MAX_REQS + 1, dtype=torch.int32, device=dev)
    with pytest.raises(B.AvmpError, match="fixed in-library scratch"):
        ctx.gather_kv_static(0, big, B.AVMP_STATIC_GATHER_MAX_REQS + 1, big, big, 0, big)
    with pytest.raises(B.AvmpError, match="invalid argument"):
        ctx.gather_kv_static(0, big, 65, big, big, 0, big)
    ctx.close()


@pytest.mark.parametrize("n_list", [1025, 1700, 2048])
def test_static_scratch_gather_long_lists(n_list):
    """Lists longer than one planning window of 1024 entries (the running sums are carried from window
    to window), twice in a row with different lists: the regular entry point (which plans such lists
    with a kernel of its own) and the oracle give the same rows."""
    import torch
    from oracle.avmp_oracle import Oracle
    from paper_2605_22416_b200 import binding as B

    dev = torch.device("cuda:0")
    m = W.PR1_MODEL
    kw = dict(max_requests=2048, max_pages=40)
    ctx = B.Context(m, 64 * W.MiB, 0.5, 8, device=dev, **kw)
    o = Oracle(m, 64 * W.MiB, 0.5, 8, with_store=True, **kw)
    lens = np.array([3, 16, 40, 1, 95, 17, 64, 33], np.uint32)
    n = len(lens)
    st = np.zeros(n, np.uint32)
    ops = W.make_ops(W.OP_ADMIT, np.arange(n) * 5, lens)          # slots 0, 5, 10, ...
    ctx.step_host(ops, n, st)
    assert np.array_equal(st, o.step(ops)) and (st == 0).all()
    rng = np.random.default_rng(n_list)
    tot = int(lens.sum())
    held = torch.from_numpy((np.arange(n) * 5).astype(np.int32)).to(dev)
    for layer in (0, 2):
        kb = rng.integers(0, 256, (tot, m.kv_row_bytes), dtype=np.uint8)
        vb = rng.integers(0, 256, (tot, m.kv_row_bytes), dtype=np.uint8)
        ctx.scatter_kv(layer, held, None, n, torch.from_numpy(kb).to(dev), torch.from_numpy(vb).to(dev))
        assert o.scatter_kv(layer, np.arange(n) * 5, np.zeros(n, np.uint32), kb, vb) == 0
    for rep, layer in enumerate((0, 2)):
        reqs = (rng.integers(0, n, n_list) * 5).astype(np.uint32)
        reqs[rng.integers(0, n_list, 7)] = 1001 + rep                 # a few empty slots in between
        total = int(o.tables()["req_len"][reqs].sum())
        cu = _three_way(ctx, o, m, dev, layer, reqs, total)
        assert cu[-1] == total
    ctx.clear_error()
    ctx.close()

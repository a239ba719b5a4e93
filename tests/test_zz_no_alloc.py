"""owl_tree_accept_static, the acceptance entry point for callers that may not allocate device
memory (a server whose allocator already owns the whole GPU, a plug-in inside a host's budget):
called through the C ABI, it must give exactly what owl_tree_accept gives, on two calls in a row
that share the library's fixed scratch array, and must refuse sizes beyond that array.

This file sorts last so that a run stopping at the first failure has already run every other test."""
import numpy as np
import pytest
import torch

from paper_2510_07535_b200 import OwlContext, make_dims, owl_tree_accept_static, workloads as W
from paper_2510_07535_b200.binding import STATIC_MAX_KEYS
from paper_2510_07535_b200.runner import DeviceWorkload, dims_of

pytestmark = pytest.mark.gpu


def _outputs(dw):
    return [t.clone() for t in (dw.accept_len, dw.accept_path, dw.bonus_token, dw.node_argmax)]


def _clear(dw):
    for t in (dw.accept_len, dw.accept_path, dw.bonus_token, dw.node_argmax):
        t.fill_(-7)


def test_static_scratch_matches_context_entry_point_twice():
    # two different batches back to back: the second call finds the first call's keys in the array
    specs = [W.config_spec(4, ctx_div=4096),                                   # 16 ragged sequences, full vocabulary
             W.Spec("na", 8, 2, [40, 50, 60], [("tree", 33, 6), ("chain", 5), ("tree", 12, 4)], seed=91, vocab=30001)]
    status = torch.full((1,), 123, dtype=torch.int32, device="cuda")
    for spec in specs:
        wl = W.generate(spec)
        dw = DeviceWorkload.upload(wl)
        ctx = OwlContext(dims_of(wl))
        _clear(dw)
        dw.accept(ctx)
        assert ctx.owl_get_status() == 0
        want = _outputs(dw)
        ctx.close()
        for _ in range(2):
            _clear(dw)
            rc = owl_tree_accept_static(dw.dims, dw.logits, dw.draft_tokens, dw.node_offsets, dw.tree_parent,
                                        dw.accept_len, dw.accept_path, dw.bonus_token, dw.node_argmax, status)
            assert rc == 0
            torch.cuda.synchronize()
            assert int(status.item()) == 0
            for got, ref in zip(_outputs(dw), want):      # integer results: bit-exact
                assert torch.equal(got, ref)


def test_static_scratch_reports_a_malformed_tree_and_recovers():
    wl = W.generate(W.Spec("na_bad", 8, 2, [30, 30], [("tree", 8, 3), ("chain", 4)], seed=92, vocab=777))
    dw = DeviceWorkload.upload(wl)
    good_parent = dw.tree_parent.clone()
    bad = good_parent.clone()
    bad[8 + 1] = 2                                        # second sequence: parent[1] = 2 >= 1
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    _clear(dw)
    rc = owl_tree_accept_static(dw.dims, dw.logits, dw.draft_tokens, dw.node_offsets, bad, dw.accept_len,
                                dw.accept_path, dw.bonus_token, None, status)
    torch.cuda.synchronize()
    assert rc == 0 and int(status.item()) == -4
    assert int(dw.accept_len[1].item()) == -7             # offending sequence left unwritten
    assert int(dw.accept_len[0].item()) >= 1
    rc = owl_tree_accept_static(dw.dims, dw.logits, dw.draft_tokens, dw.node_offsets, good_parent, dw.accept_len,
                                dw.accept_path, dw.bonus_token, None, status)
    torch.cuda.synchronize()
    assert rc == 0 and int(status.item()) == 0            # the call cleared the status word itself


def test_static_scratch_survives_inconsistent_offsets():
    """A call whose node_offsets do not describe its rows leaves progress counters dirty in the shared array; the
    calls after it (a smaller batch first) must still agree with the context entry point."""
    big = W.generate(W.Spec("na_offs", 8, 2, [30] * 4, [("tree", 8, 3), ("chain", 4)] * 2, seed=93, vocab=20000))
    small = W.generate(W.Spec("na_offs2", 8, 2, [30], [("tree", 9, 3)], seed=94, vocab=20000))
    want = {}
    for name, wl in (("big", big), ("small", small)):
        dw = DeviceWorkload.upload(wl)
        ctx = OwlContext(dims_of(wl))
        dw.accept(ctx)
        assert ctx.owl_get_status() == 0
        want[name] = (dw, _outputs(dw))
        ctx.close()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    dw_big = want["big"][0]
    bad_offsets = torch.tensor([0, 8, 8, 20, 24], dtype=torch.int32, device="cuda")     # sequence 1 has no nodes
    rc = owl_tree_accept_static(dw_big.dims, dw_big.logits, dw_big.draft_tokens, bad_offsets, dw_big.tree_parent,
                                dw_big.accept_len, dw_big.accept_path, dw_big.bonus_token, None, status)
    torch.cuda.synchronize()
    assert rc == 0 and int(status.item()) == -4
    for name in ("small", "big", "small", "big"):
        dw, ref = want[name]
        _clear(dw)
        rc = owl_tree_accept_static(dw.dims, dw.logits, dw.draft_tokens, dw.node_offsets, dw.tree_parent,
                                    dw.accept_len, dw.accept_path, dw.bonus_token, dw.node_argmax, status)
        torch.cuda.synchronize()
        assert rc == 0 and int(status.item()) == 0
        for got, r in zip(_outputs(dw), ref):
            assert torch.equal(got, r)


def test_static_scratch_rejects_sizes_beyond_the_array():
    V = 128256
    chunks = (V + 8191) // 8192
    n = STATIC_MAX_KEYS // chunks + 1                    # 1025 rows = 25 sequences of 41 nodes
    assert n % 25 == 0
    d = make_dims(batch=25, total_nodes=n, max_nodes=n // 25, vocab=V)
    one = torch.zeros(1, dtype=torch.int32, device="cuda")
    lg = torch.zeros(1, dtype=torch.float32, device="cuda")
    # nothing is launched, so the (too small) buffers are never touched
    rc = owl_tree_accept_static(d, lg, one, None, one, one, one, one, None, None, check=False)
    assert rc == -7

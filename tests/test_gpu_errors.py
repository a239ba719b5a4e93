"""Error behaviour of the C ABI: host-detectable errors launch nothing; device-detected errors set
the status word, leave the offending sequence's outputs untouched and do not disturb the others."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2510_07535_b200 import OwlContext, OwlError, make_dims, workloads as W
from paper_2510_07535_b200.runner import DeviceWorkload, dims_of

pytestmark = pytest.mark.gpu


def _wl():
    return W.generate(W.Spec("err", 8, 2, [200, 150, 90], [("tree", 8, 3), ("chain", 4), ("tree", 6, 3)],
                             shuffle_pages=True, seed=5, vocab=512))


def test_host_detected_errors():
    wl = _wl()
    dw = DeviceWorkload.upload(wl)
    ctx = OwlContext(dims_of(wl))
    n0 = ctx.launch_count()
    bad = dims_of(wl); bad.head_dim = 64
    assert DeviceWorkload.attn(dataclass_replace(dw, dims=bad), ctx, check=False) == -2
    bad = dims_of(wl); bad.max_nodes = 65
    assert DeviceWorkload.attn(dataclass_replace(dw, dims=bad), ctx, check=False) == -2
    bad = dims_of(wl); bad.num_kv_heads = 3
    assert DeviceWorkload.attn(dataclass_replace(dw, dims=bad), ctx, check=False) == -1
    bad = dims_of(wl); bad.batch = 0
    assert DeviceWorkload.attn(dataclass_replace(dw, dims=bad), ctx, check=False) == -1
    bad = dims_of(wl); bad.batch = 9
    assert DeviceWorkload.attn(dataclass_replace(dw, dims=bad), ctx, check=False) in (-1, -7)
    bad = dims_of(wl); bad.path_stride = 4
    assert DeviceWorkload.accept(dataclass_replace(dw, dims=bad), ctx, check=False) == -1
    assert DeviceWorkload.attn(dataclass_replace(dw, q=None), ctx, check=False) == -1
    assert DeviceWorkload.accept(dataclass_replace(dw, logits=None), ctx, check=False) == -1
    with pytest.raises(OwlError):
        DeviceWorkload.attn(dataclass_replace(dw, q=None), ctx)
    assert ctx.launch_count() == n0          # nothing was launched
    assert ctx.owl_get_status() == 0
    ctx.close()


def dataclass_replace(dw, **kw):
    import dataclasses
    return dataclasses.replace(dw, **kw)


def test_create_rejects_bad_device_and_dims():
    with pytest.raises(OwlError):
        OwlContext(make_dims(batch=1, total_nodes=1, max_nodes=1, num_q_heads=8, num_kv_heads=2, head_dim=96,
                             max_pages_per_seq=4, num_pages=4))
    with pytest.raises(OwlError):
        OwlContext(make_dims(batch=2000, total_nodes=2000, max_nodes=1, vocab=10))


def test_too_large_for_context():
    wl = _wl()
    small = dims_of(wl); small.batch = 1; small.total_nodes = 8
    ctx = OwlContext(small)
    dw = DeviceWorkload.upload(wl)
    assert dw.attn(ctx, check=False) == -7
    assert dw.accept(ctx, check=False) == -7
    ctx.close()


def test_bad_tree_is_reported_and_isolated():
    wl = _wl()
    ref_out, _ = oracle.verify_attn(wl.q, wl.k_cache, wl.v_cache, wl.block_table, wl.ctx_lens, wl.node_offsets,
                                    wl.tree_parent, wl.sm_scale)
    r_alen, r_path, r_bonus, _ = oracle.tree_accept(wl.logits, wl.draft_tokens, wl.node_offsets, wl.tree_parent, 64)
    bad = wl.tree_parent.copy()
    bad[8 + 2] = 3                      # sequence 1 (nodes 8..11): parent[2] = 3 >= 2
    dw = DeviceWorkload.upload(wl)
    dw.tree_parent = torch.from_numpy(bad).cuda()
    ctx = OwlContext(dims_of(wl))
    dw.out.fill_(7.0); dw.accept_len.fill_(-5)
    dw.attn(ctx)
    assert ctx.owl_get_status() == -4
    out = dw.out_f32()
    assert np.all(out[8:12] == 7.0)                             # offending sequence untouched
    assert np.abs(out[:8] - ref_out[:8]).max() <= 1e-2          # the others are right
    assert np.abs(out[12:] - ref_out[12:]).max() <= 1e-2
    dw.accept(ctx)
    assert ctx.owl_get_status() == -4
    alen = dw.accept_len.cpu().numpy()
    assert alen[1] == -5 and alen[0] == r_alen[0] and alen[2] == r_alen[2]
    assert ctx.owl_get_status() == 0                            # reading the status clears it
    # the whole step in one call (scan and walk inside the attention kernels): same verdict, same isolation
    dw.out.fill_(7.0); dw.accept_len.fill_(-5)
    dw.step(ctx)
    assert ctx.owl_get_status() == -4
    out = dw.out_f32()
    assert np.all(out[8:12] == 7.0)
    assert np.abs(out[:8] - ref_out[:8]).max() <= 1e-2 and np.abs(out[12:] - ref_out[12:]).max() <= 1e-2
    alen = dw.accept_len.cpu().numpy()
    assert alen[1] == -5 and alen[0] == r_alen[0] and alen[2] == r_alen[2]
    # the context stays usable
    dw2 = DeviceWorkload.upload(wl)
    dw2.step(ctx)
    assert ctx.owl_get_status() == 0
    np.testing.assert_array_equal(dw2.accept_len.cpu().numpy(), r_alen)
    assert np.abs(dw2.out_f32() - ref_out).max() <= 1e-2
    ctx.close()


def test_bad_page_is_reported_and_isolated():
    wl = _wl()
    ref_out, _ = oracle.verify_attn(wl.q, wl.k_cache, wl.v_cache, wl.block_table, wl.ctx_lens, wl.node_offsets,
                                    wl.tree_parent, wl.sm_scale)
    dw = DeviceWorkload.upload(wl)
    bt = wl.block_table.copy()
    bt[2, 1] = wl.num_pages + 3          # sequence 2: a page id past the cache
    dw.block_table = torch.from_numpy(bt).cuda()
    ctx = OwlContext(dims_of(wl))
    dw.out.fill_(7.0)
    dw.attn(ctx)
    assert ctx.owl_get_status() == -5
    out = dw.out_f32()
    assert np.all(out[12:] == 7.0)
    assert np.abs(out[:12] - ref_out[:12]).max() <= 1e-2
    # a context length that does not fit the block table is a page error too
    dw = DeviceWorkload.upload(wl)
    cl = wl.ctx_lens.copy(); cl[0] = wl.max_pages_per_seq * 16
    dw.ctx_lens = torch.from_numpy(cl).cuda()
    dw.out.fill_(7.0)
    dw.attn(ctx)
    assert ctx.owl_get_status() == -5
    out = dw.out_f32()
    assert np.all(out[:8] == 7.0) and np.abs(out[8:] - ref_out[8:]).max() <= 1e-2
    ctx.close()


def test_scale_and_head_limits():
    wl = _wl()
    dw = DeviceWorkload.upload(wl)
    ctx = OwlContext(dims_of(wl))
    n0 = ctx.launch_count()
    for bad_scale in (0.0, -0.5, float("nan"), float("inf")):
        bad = dims_of(wl); bad.sm_scale = bad_scale
        assert DeviceWorkload.attn(dataclass_replace(dw, dims=bad), ctx, check=False) == -1
    bad = dims_of(wl); bad.num_q_heads = 512; bad.num_kv_heads = 256
    assert DeviceWorkload.attn(dataclass_replace(dw, dims=bad), ctx, check=False) == -2
    assert ctx.launch_count() == n0
    ctx.close()


def test_bounded_wait_gives_up_and_reports_timeout():
    """The kernels' wait routine on a barrier nothing completes: gives up after the limit, reports
    OWL_ERR_TIMEOUT, a second wait returns at once, and the next ordinary call on the context is clean."""
    wl = _wl()
    dw = DeviceWorkload.upload(wl)
    ctx = OwlContext(dims_of(wl))
    limit = 1_000_000                                   # 1 ms
    st, first_ns, second_ns = ctx.owl_selftest_wait(limit)
    assert st == -6
    assert limit <= first_ns <= 50 * limit              # gave up after the limit, and soon after it
    assert second_ns < limit // 2                       # abort flag up: no second spin
    assert ctx.owl_get_status() == 0                    # reading the status cleared it
    assert ctx.lib.owl_selftest_wait(ctx._h, 0, None, None) == -1          # limit out of range: nothing launched
    assert ctx.lib.owl_selftest_wait(ctx._h, 2_000_000_000, None, None) == -1
    dw.step(ctx)
    assert ctx.owl_get_status() == 0
    ref_out, _ = oracle.verify_attn(wl.q, wl.k_cache, wl.v_cache, wl.block_table, wl.ctx_lens, wl.node_offsets,
                                    wl.tree_parent, wl.sm_scale)
    assert np.abs(dw.out_f32() - ref_out).max() <= 1e-2
    ctx.close()


def _accept_equals_oracle(dw, wl):
    alen, path, bonus, am = oracle.tree_accept(wl.logits, wl.draft_tokens, wl.node_offsets, wl.tree_parent, 64)
    np.testing.assert_array_equal(dw.node_argmax.cpu().numpy(), am)
    np.testing.assert_array_equal(dw.accept_len.cpu().numpy(), alen)
    np.testing.assert_array_equal(dw.accept_path.cpu().numpy(), path)
    np.testing.assert_array_equal(dw.bonus_token.cpu().numpy(), bonus)


def test_inconsistent_node_offsets_are_reported_and_leave_no_trace():
    """Offsets that do not describe the call's rows (a sequence with no nodes, a total that is not total_nodes) set
    the status word; the per-sequence progress counters they leave dirty must not disturb later calls, also
    when those have a smaller batch."""
    big = W.generate(W.Spec("offs", 8, 2, [40] * 6, [("tree", 8, 3), ("chain", 4), ("tree", 6, 3)] * 2, seed=15, vocab=20000))
    small = W.generate(W.Spec("offs2", 8, 2, [40] * 2, [("chain", 5), ("tree", 7, 3)], seed=16, vocab=20000))
    ctx = OwlContext(dims_of(big))
    dw_big, dw_small = DeviceWorkload.upload(big), DeviceWorkload.upload(small)
    for bad_offsets in ([0, 8, 8, 18, 26, 30, 36],          # sequence 1 has no nodes
                        [0, 8, 12, 18, 26, 30, 35],         # last offset is not total_nodes
                        [2, 8, 12, 18, 26, 30, 36]):        # first offset is not 0
        bad = dataclass_replace(dw_big, node_offsets=torch.tensor(bad_offsets, dtype=torch.int32, device="cuda"))
        bad.accept(ctx)
        assert ctx.owl_get_status() == -4
        for dw, wl in ((dw_small, small), (dw_big, big), (dw_small, small), (dw_big, big)):
            for t in (dw.accept_len, dw.accept_path, dw.bonus_token, dw.node_argmax):
                t.fill_(-9)
            dw.accept(ctx)
            assert ctx.owl_get_status() == 0
            _accept_equals_oracle(dw, wl)
    ctx.close()

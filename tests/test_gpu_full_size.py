"""Parity at the benchmark's full sizes, in the launch configuration bench.py times: the CUDA path
runs the whole configuration; the oracle recomputes a seeded sample of (node, head) output rows one
by one, and the whole acceptance (arg-max over the full vocabulary is cheap on the CPU)."""
import numpy as np
import pytest

import oracle
from paper_2510_07535_b200 import OwlContext, workloads as W
from paper_2510_07535_b200.runner import DeviceWorkload, dims_of

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("idx", [0, 1, 2, 3, 4])
def test_full_configuration_sampled_rows(idx):
    wl = W.generate(W.config_spec(idx))
    dw = DeviceWorkload.upload(wl)
    ctx = OwlContext(dims_of(wl))
    dw.step(ctx)
    assert ctx.owl_get_status() == 0
    N, Hq, _ = wl.q.shape
    rng = np.random.default_rng(100 + idx)
    n_rows = 64
    # every sequence contributes rows, including its last node (deepest mask) and its root
    nodes = np.concatenate([rng.integers(0, N, size=n_rows - 2 * wl.spec.batch),
                            wl.node_offsets[:-1], wl.node_offsets[1:] - 1]).astype(np.int32)
    heads = rng.integers(0, Hq, size=len(nodes)).astype(np.int32)
    ref_out, ref_lse = oracle.verify_attn(wl.q, wl.k_cache, wl.v_cache, wl.block_table, wl.ctx_lens,
                                          wl.node_offsets, wl.tree_parent, wl.sm_scale, rows=(nodes, heads))
    out = dw.out_f32()[nodes, heads]
    lse = dw.lse.cpu().numpy()[nodes, heads]
    assert np.abs(out - ref_out).max() <= 1e-2
    assert np.abs(lse - ref_lse).max() <= 1e-3
    # properties that hold at any size, on every row
    all_lse = dw.lse.cpu().numpy()
    assert np.all(np.isfinite(all_lse)) and np.all(np.isfinite(dw.out_f32()))
    alen, path, bonus, am = oracle.tree_accept(wl.logits, wl.draft_tokens, wl.node_offsets, wl.tree_parent, 64)
    np.testing.assert_array_equal(dw.node_argmax.cpu().numpy(), am)
    np.testing.assert_array_equal(dw.accept_len.cpu().numpy(), alen)
    np.testing.assert_array_equal(dw.accept_path.cpu().numpy(), path)
    np.testing.assert_array_equal(dw.bonus_token.cpu().numpy(), bonus)
    ctx.close()

"""The routed (hybrid) batch and the fp16 variant on the GPU, through the C ABI, against the CPU oracle:
Algorithm 1's routing, Prepare(d) on a routed batch, verify attention with fp16 caches."""
import json
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2510_07535_b200 import OwlContext, make_dims, owl_howl_route, workloads as W
from paper_2510_07535_b200.runner import dims_of

pytestmark = pytest.mark.gpu

DEV = "cuda"
dev_i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(DEV)


def test_routing_matches_the_trace_and_the_oracle(golden_dir):
    g = json.load(open(os.path.join(golden_dir, "howl_routing_trace.json")))
    state = np.zeros(1, np.uint8)
    for score, route, after in zip(g["scores"], g["routes"], g["lastwaslinear_after"]):
        assert owl_howl_route(np.array([score], np.float32), g["c"], state).tolist() == [route]
        assert state.tolist() == [after]
    rng = np.random.default_rng(2)
    a, b = np.zeros(64, np.uint8), np.zeros(64, np.uint8)
    for step in range(200):
        score = rng.choice([0.5, 8.0, 9.0, 9.25, 100.0, np.inf], size=64).astype(np.float32)
        np.testing.assert_array_equal(owl_howl_route(score, 9.0, a), oracle.howl_route(score, 9.0, b))
        np.testing.assert_array_equal(a, b)
    # a NaN score is no reason to skip the tree drafter; a NaN threshold is an error
    assert owl_howl_route(np.array([np.nan], np.float32), 9.0, np.zeros(1, np.uint8)).tolist() == [2]
    with pytest.raises(Exception):
        owl_howl_route(np.array([1.0], np.float32), float("nan"), np.zeros(1, np.uint8))


def test_prepare_hybrid_matches_oracle():
    rng = np.random.default_rng(3)
    ctx = OwlContext(make_dims(batch=8, total_nodes=8 * 64, max_nodes=64))
    for trial in range(25):
        B = int(rng.integers(1, 9))
        route = rng.integers(0, 3, size=B).astype(np.int32)
        parents = [W.chain_parents(int(rng.integers(1, 65))) if route[b] == 0 else W.random_tree_parents(rng, int(rng.integers(1, 33)), 8)
                   for b in range(B)]
        counts = np.array([len(p) for p in parents])
        offs = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
        par = np.concatenate(parents).astype(np.int32)
        tok = rng.integers(0, 128256, size=len(par)).astype(np.int32)
        lens = rng.integers(0, 131072, size=B).astype(np.int32)
        N = len(par)
        d = make_dims(batch=B, total_nodes=N, max_nodes=int(counts.max()))
        outs = [torch.full((B + 1,), -7, dtype=torch.int32, device=DEV)] + [torch.full((2 * N,), -7, dtype=torch.int32, device=DEV) for _ in range(4)]
        ctx.owl_prepare_hybrid(d, dev_i32(offs), dev_i32(par), dev_i32(tok), dev_i32(lens), dev_i32(route), 128255, *outs)
        assert ctx.owl_get_status() == 0
        ref = oracle.prepare_hybrid(offs, par, tok, lens, route, 128255)
        M = int(ref[0][-1])
        np.testing.assert_array_equal(outs[0].cpu().numpy(), ref[0])
        for got, r in zip(outs[1:], ref[1:]):
            np.testing.assert_array_equal(got.cpu().numpy()[:M], r)
            assert np.all(got.cpu().numpy()[M:] == -7)
    # a 33-node tree on a tree route cannot get its leaves (66 nodes): reported, unwritten; its neighbour is prepared
    par = np.concatenate([W.chain_parents(33), W.chain_parents(5)]).astype(np.int32)
    offs, tok = np.array([0, 33, 38], np.int32), np.arange(38, dtype=np.int32)
    d = make_dims(batch=2, total_nodes=38, max_nodes=33)
    outs = [torch.full((3,), -7, dtype=torch.int32, device=DEV)] + [torch.full((76,), -7, dtype=torch.int32, device=DEV) for _ in range(4)]
    ctx.owl_prepare_hybrid(d, dev_i32(offs), dev_i32(par), dev_i32(tok), dev_i32([7, 9]), dev_i32([2, 2]), 5, *outs)
    assert ctx.owl_get_status() == -4
    assert np.all(outs[1].cpu().numpy()[:66] == -7)
    ref = oracle.prepare_spec_tree(np.array([0, 5], np.int32), par[33:], tok[33:], np.array([9], np.int32), 5)
    np.testing.assert_array_equal(outs[1].cpu().numpy()[66:76], ref[1])
    ctx.close()


def _f16_workload(spec):
    wl = W.generate(spec)
    for name in ("q", "k_cache", "v_cache"):
        setattr(wl, name, W.bf16_bits_to_f32(getattr(wl, name)).astype(np.float16).view(np.uint16))
    return wl


def check_attention_f16(wl):
    h = lambda bits: torch.from_numpy(np.ascontiguousarray(bits).view(np.float16)).to(DEV)
    N, Hq, D = wl.q.shape
    d = dims_of(wl)
    ctx = OwlContext(d)
    out = torch.zeros((N, Hq, D), dtype=torch.float16, device=DEV)
    lse = torch.zeros((N, Hq), dtype=torch.float32, device=DEV)
    args = (d, h(wl.q), h(wl.k_cache), h(wl.v_cache), dev_i32(wl.block_table), dev_i32(wl.ctx_lens), dev_i32(wl.node_offsets),
            dev_i32(wl.tree_parent))
    ctx.owl_verify_attn_f16(*args, out, lse)
    assert ctx.owl_get_status() == 0
    ref_out, ref_lse = oracle.verify_attn(wl.q, wl.k_cache, wl.v_cache, wl.block_table, wl.ctx_lens, wl.node_offsets,
                                          wl.tree_parent, wl.sm_scale, dtype="f16")
    eo = np.abs(out.float().cpu().numpy().astype(np.float64) - ref_out).max()
    el = np.abs(lse.cpu().numpy().astype(np.float64) - ref_lse).max()
    out1, lse1 = out.clone(), lse.clone()
    out.zero_(); lse.zero_()
    ctx.owl_verify_attn_f16(*args, out, lse)
    assert torch.equal(out1, out) and torch.equal(lse1, lse)           # run to run bit-identical
    ctx.close()
    assert eo <= 1e-2 and el <= 1e-3, (eo, el)


@pytest.mark.parametrize("idx,div", [(0, 4), (1, 32), (2, 128), (3, 64), (4, 64)])
def test_scaled_down_configs_attention_f16(idx, div):
    spec = W.config_spec(idx, ctx_div=div, vocab=1024)
    spec.with_logits = False
    check_attention_f16(_f16_workload(spec))


@pytest.mark.parametrize("hq,hkv,trees,ctx,page", [
    (8, 2, [("chain", 1)], [0], 16),
    (4, 1, [("tree", 64, 8)], [0], 16),
    (32, 8, [("tree", 64, 8), ("chain", 3)], [777, 15], 16),
    (12, 4, [("tree", 11, 4), ("chain", 7)], [300, 1000], 64),
])
def test_edge_shapes_attention_f16(hq, hkv, trees, ctx, page):
    check_attention_f16(_f16_workload(W.Spec("edge16", hq, hkv, ctx, trees, shuffle_pages=True, page_size=page,
                                             seed=hq * 100 + ctx[0], with_logits=False)))


def test_many_sequences_f16():
    rng = np.random.default_rng(7)
    ctx = [int(x) for x in rng.integers(1, 300, size=40)]
    trees = [[("tree", 64, 8), ("chain", 3), ("tree", 17, 4)][int(rng.integers(0, 3))] for _ in range(40)]
    check_attention_f16(_f16_workload(W.Spec("many16", 16, 4, ctx, trees, shuffle_pages=True, seed=71, with_logits=False)))

"""Pins (CPU only) of the oracle's routing (Algorithm 1), of Prepare(d) on a routed batch, and of the fp16
reading of the attention inputs (the paper's data type)."""
import json
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2510_07535_b200 import workloads as W


def test_routing_follows_the_hand_worked_trace(golden_dir):
    g = json.load(open(os.path.join(golden_dir, "howl_routing_trace.json")))
    state = np.zeros(1, np.uint8)
    for score, route, after in zip(g["scores"], g["routes"], g["lastwaslinear_after"]):
        assert oracle.howl_route(np.array([score], np.float32), g["c"], state).tolist() == [route]
        assert state.tolist() == [after]


def test_routing_state_machine_properties():
    """Sequences are routed independently; a tree step right after a linear one uses D_nospec exactly once;
    with every score at or below c (c = the longest acceptance a depth-8 tree allows, 9) nothing is ever linear."""
    rng = np.random.default_rng(1)
    B, c = 16, 9.0
    state = np.zeros(B, np.uint8)
    prev = np.full(B, 2)
    for step in range(300):
        score = rng.choice([1.0, 5.0, 9.0, 9.5, 30.0], size=B).astype(np.float32)
        route = oracle.howl_route(score, c, state)
        assert np.array_equal(route == 0, score > c)
        tree = route != 0
        assert np.all(route[tree & (prev == 0)] == 1) and np.all(route[tree & (prev != 0)] == 2)
        assert np.array_equal(state, (route == 0).astype(np.uint8))
        prev = route
    state = np.zeros(B, np.uint8)
    for step in range(20):
        assert np.all(oracle.howl_route(rng.uniform(1, 9, size=B).astype(np.float32), c, state) == 2)


def test_hybrid_prepare_is_prepare_per_sequence():
    rng = np.random.default_rng(2)
    for trial in range(30):
        B = int(rng.integers(1, 7))
        route = rng.integers(0, 3, size=B).astype(np.int32)
        parents = [W.chain_parents(int(rng.integers(1, 41))) if route[b] == 0 else W.random_tree_parents(rng, int(rng.integers(1, 33)), 8)
                   for b in range(B)]
        counts = np.array([len(p) for p in parents])
        offs = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
        par = np.concatenate(parents).astype(np.int32)
        tok = rng.integers(0, 1000, size=len(par)).astype(np.int32)
        ctx = rng.integers(0, 5000, size=B).astype(np.int32)
        o, p, d, ids, pos = oracle.prepare_hybrid(offs, par, tok, ctx, route, 4242)
        assert o[0] == 0 and len(p) == o[-1]
        for b in range(B):
            n = int(counts[b])
            sl_in = slice(int(offs[b]), int(offs[b + 1]))
            one = oracle.prepare_spec_tree(np.array([0, n], np.int32), par[sl_in], tok[sl_in], ctx[b:b + 1], 4242)
            take = n if route[b] == 0 else 2 * n          # a linear sequence keeps its chain, without any [SPEC]
            assert o[b + 1] - o[b] == take
            sl = slice(int(o[b]), int(o[b + 1]))
            for got, ref in zip((p, d, ids, pos), one[1:]):
                assert np.array_equal(got[sl], ref[:take])
            if route[b] == 0:
                assert np.all(d[sl][1:] >= 0) and np.array_equal(pos[sl], ctx[b] + np.arange(n))   # plain text positions


# ----------------------------------------------------------------------------- fp16 inputs

def test_decoders_agree_with_library_conversions_on_every_bit_pattern():
    bits = np.arange(65536, dtype=np.uint16)
    ref16 = bits.view(np.float16).astype(np.float64)                       # numpy's IEEE binary16
    got16 = oracle.decode16(bits, "f16")
    assert np.array_equal(np.isnan(ref16), np.isnan(got16)) and np.array_equal(ref16[~np.isnan(ref16)], got16[~np.isnan(ref16)])
    assert np.array_equal(np.signbit(ref16), np.signbit(got16))
    refb = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).double().numpy()   # torch's bfloat16
    gotb = oracle.decode16(bits, "bf16")
    assert np.array_equal(np.isnan(refb), np.isnan(gotb)) and np.array_equal(refb[~np.isnan(refb)], gotb[~np.isnan(refb)])


def _as_f16(wl):
    """The same workload with q / K / V re-encoded as fp16 bit patterns (nearest fp16 of the bf16 draws)."""
    for name in ("q", "k_cache", "v_cache"):
        x = W.bf16_bits_to_f32(getattr(wl, name))
        setattr(wl, name, x.astype(np.float16).view(np.uint16))
    return wl


@pytest.mark.parametrize("trees,ctx,hq,hkv", [([("tree", 9, 3)], [37], 8, 2), ([("chain", 5), ("tree", 20, 5)], [0, 50], 4, 4)])
def test_f16_attention_against_dense_brute_force(trees, ctx, hq, hkv):
    wl = _as_f16(W.generate(W.Spec("f16", hq, hkv, ctx, trees, shuffle_pages=True, seed=9, with_logits=False), threads=1))
    out, lse = oracle.verify_attn(wl.q, wl.k_cache, wl.v_cache, wl.block_table, wl.ctx_lens, wl.node_offsets,
                                  wl.tree_parent, wl.sm_scale, dtype="f16")
    G = hq // hkv
    f = lambda bits: bits.view(np.float16).astype(np.float64)
    for b in range(len(ctx)):
        lo, hi = int(wl.node_offsets[b]), int(wl.node_offsets[b + 1])
        n, L = hi - lo, int(wl.ctx_lens[b])
        par = wl.tree_parent[lo:hi]
        anc = np.eye(n, dtype=bool)
        for i in range(n):                                   # ancestors by the recursion anc[i] = anc[parent] | {i}
            if par[i] >= 0:
                anc[i] |= anc[par[i]]
        vis = np.concatenate([np.ones((n, L), bool), anc], axis=1)
        pos = np.arange(L + n)
        pages = wl.block_table[b, pos // wl.spec.page_size]
        for h_q in range(hq):
            K = f(wl.k_cache[pages, h_q // G, pos % wl.spec.page_size])
            V = f(wl.v_cache[pages, h_q // G, pos % wl.spec.page_size])
            S = np.where(vis, wl.sm_scale * (f(wl.q[lo:hi, h_q]) @ K.T), -np.inf)
            P = np.exp(S - S.max(axis=1, keepdims=True))
            assert np.allclose(out[lo:hi, h_q], (P / P.sum(axis=1, keepdims=True)) @ V, rtol=0, atol=1e-12)
            assert np.allclose(lse[lo:hi, h_q], np.log(P.sum(axis=1)) + S.max(axis=1), rtol=0, atol=1e-12)


def test_f16_and_bf16_readings_agree_on_values_both_can_hold():
    """The same real inputs, once as bf16 patterns and once as fp16 patterns, give the same attention."""
    wl = W.generate(W.Spec("both", 8, 2, [70, 3], [("tree", 12, 4), ("chain", 4)], shuffle_pages=True, seed=10, with_logits=False), threads=1)
    for name in ("q", "k_cache", "v_cache"):          # bf16 values below fp16's normal range have no fp16 twin: drop them
        x = W.bf16_bits_to_f32(getattr(wl, name))
        x[np.abs(x) < 2.0 ** -14] = 0.0
        setattr(wl, name, W.f32_to_bf16_bits(x).reshape(x.shape))
    a = oracle.verify_attn(wl.q, wl.k_cache, wl.v_cache, wl.block_table, wl.ctx_lens, wl.node_offsets, wl.tree_parent, wl.sm_scale)
    wl = _as_f16(wl)
    b = oracle.verify_attn(wl.q, wl.k_cache, wl.v_cache, wl.block_table, wl.ctx_lens, wl.node_offsets, wl.tree_parent, wl.sm_scale,
                           dtype="f16")
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
    # and reading fp16 patterns as bf16 is a different problem: the switch is not ignored
    c = oracle.verify_attn(wl.q, wl.k_cache, wl.v_cache, wl.block_table, wl.ctx_lens, wl.node_offsets, wl.tree_parent, wl.sm_scale)
    assert not np.allclose(a[0], c[0])

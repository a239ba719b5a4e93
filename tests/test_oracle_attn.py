"""Pins for the attention oracle (CPU only).

Each test checks ``oracle.verify_attn`` against something other than itself: a dense
brute force written a different way, a library routine on a special case, the
paper's worked mask example, or an invariant of softmax attention.
"""
import json
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2510_07535_b200 import workloads as W


def _f64(bits):
    return W.bf16_bits_to_f32(bits).astype(np.float64)


def _gather_kv(cache, block_table, b, h, length, page):
    """Logical [length, D] view of one sequence/head from the paged cache."""
    pos = np.arange(length)
    pages = block_table[b, pos // page]
    return _f64(cache[pages, h, pos % page])


def _dense_mask(parent):
    """Ancestor-or-self relation by transitive closure of the child->parent edges
    (boolean matrix powers), deliberately not by pointer chasing."""
    n = len(parent)
    E = np.zeros((n, n), dtype=bool)
    for i, p in enumerate(parent):
        if p >= 0:
            E[i, p] = True
    R = np.eye(n, dtype=bool)
    step = np.eye(n, dtype=bool)
    for _ in range(n):
        step = (step.astype(np.int64) @ E.astype(np.int64)) > 0
        R |= step
    return R


def brute_force(wl):
    """softmax(Q K^T * scale + mask) V with an explicit dense mask, numpy fp64."""
    sp = wl.spec
    G = sp.num_q_heads // sp.num_kv_heads
    N, Hq, D = wl.q.shape
    out = np.zeros((N, Hq, D))
    lse = np.zeros((N, Hq))
    for b in range(sp.batch):
        lo, hi = int(wl.node_offsets[b]), int(wl.node_offsets[b + 1])
        n = hi - lo
        L = int(wl.ctx_lens[b])
        vis = np.concatenate([np.ones((n, L), dtype=bool), _dense_mask(wl.tree_parent[lo:hi])], axis=1)
        for hq in range(Hq):
            h = hq // G
            K = _gather_kv(wl.k_cache, wl.block_table, b, h, L + n, sp.page_size)
            V = _gather_kv(wl.v_cache, wl.block_table, b, h, L + n, sp.page_size)
            Q = _f64(wl.q[lo:hi, hq])
            S = wl.sm_scale * (Q @ K.T)
            S = np.where(vis, S, -np.inf)
            m = S.max(axis=1, keepdims=True)
            P = np.exp(S - m)
            Z = P.sum(axis=1, keepdims=True)
            out[lo:hi, hq] = (P / Z) @ V
            lse[lo:hi, hq] = (m + np.log(Z))[:, 0]
    return out, lse


def _run(wl, rows=None):
    return oracle.verify_attn(wl.q, wl.k_cache, wl.v_cache, wl.block_table, wl.ctx_lens, wl.node_offsets,
                              wl.tree_parent, wl.sm_scale, rows=rows)


def _small(trees, ctx, hq=8, hkv=2, shuffle=True, seed=3, prescaled=True):
    return W.generate(W.Spec("tiny", hq, hkv, ctx, trees, shuffle_pages=shuffle, seed=seed,
                             with_logits=False, q_prescaled=prescaled), threads=1)


@pytest.mark.parametrize("hq,hkv", [(1, 1), (4, 1), (8, 2), (8, 1)])
def test_matches_dense_brute_force(hq, hkv):
    wl = _small([("tree", 8, 3), ("chain", 5), ("tree", 6, 2), ("chain", 1)], [37, 64, 1, 19], hq, hkv, seed=hq * 10 + hkv)
    out, lse = _run(wl)
    ref_out, ref_lse = brute_force(wl)
    np.testing.assert_allclose(out, ref_out, rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse, ref_lse, rtol=0, atol=1e-12)


def test_llama_scale_form_matches_brute_force():
    wl = _small([("tree", 7, 3)], [50], prescaled=False)
    assert abs(wl.sm_scale - 1 / np.sqrt(128)) < 1e-12
    out, lse = _run(wl)
    ref_out, ref_lse = brute_force(wl)
    np.testing.assert_allclose(out, ref_out, atol=1e-12)
    np.testing.assert_allclose(lse, ref_lse, atol=1e-12)


def test_row_subset_equals_full():
    wl = _small([("tree", 8, 3), ("chain", 4)], [33, 20])
    out, lse = _run(wl)
    rn = np.array([0, 3, 7, 8, 11], dtype=np.int32)
    rh = np.array([0, 5, 7, 2, 6], dtype=np.int32)
    o2, l2 = _run(wl, rows=(rn, rh))
    np.testing.assert_array_equal(o2, out[rn, rh])
    np.testing.assert_array_equal(l2, lse[rn, rh])


def test_single_node_is_plain_decode_attention():
    """One drafted node: ordinary one-token decode attention over L+1 keys (library SDPA, fp64)."""
    wl = _small([("chain", 1)], [83], hq=8, hkv=2, shuffle=True)
    out, lse = _run(wl)
    G = 4
    for hq in range(8):
        K = torch.from_numpy(_gather_kv(wl.k_cache, wl.block_table, 0, hq // G, 84, 16))
        V = torch.from_numpy(_gather_kv(wl.v_cache, wl.block_table, 0, hq // G, 84, 16))
        Q = torch.from_numpy(_f64(wl.q[0:1, hq]))
        ref = torch.nn.functional.scaled_dot_product_attention(Q[None], K[None], V[None], scale=wl.sm_scale)[0]
        np.testing.assert_allclose(out[0, hq], ref[0].numpy(), atol=1e-12)
        ref_lse = torch.logsumexp(wl.sm_scale * (Q @ K.T), dim=-1)
        np.testing.assert_allclose(lse[0, hq], ref_lse[0].item(), atol=1e-12)


def test_chain_is_causal_attention():
    """Chain-shaped tree: row i equals causal attention at position L+i (library SDPA is_causal, fp64)."""
    n, L = 9, 45
    wl = _small([("chain", n)], [L], hq=4, hkv=2, shuffle=True, prescaled=False)
    out, _ = _run(wl)
    for hq in range(4):
        K = torch.from_numpy(_gather_kv(wl.k_cache, wl.block_table, 0, hq // 2, L + n, 16))
        V = torch.from_numpy(_gather_kv(wl.v_cache, wl.block_table, 0, hq // 2, L + n, 16))
        # queries of the prefix positions do not matter for the last n rows: fill with zeros
        Q = torch.zeros(L + n, 128, dtype=torch.float64)
        Q[L:] = torch.from_numpy(_f64(wl.q[:, hq]))
        ref = torch.nn.functional.scaled_dot_product_attention(Q[None], K[None], V[None], is_causal=True,
                                                               scale=wl.sm_scale)[0]
        np.testing.assert_allclose(out[:, hq], ref[L:].numpy(), atol=1e-12)


def test_paper_decode_stage_mask_example(golden_dir):
    """The three paths of the 'Decode Stage' example: uniform scores + one-hot V expose the visible set."""
    with open(os.path.join(golden_dir, "decode_stage_mask_example.json")) as f:
        gold = json.load(f)
    parent = np.array(gold["tree_parent"], dtype=np.int32)
    n, L, D, P = len(parent), 5, 128, 16
    pages = (L + n + P - 1) // P
    k_cache = np.zeros((pages, 1, P, D), dtype=np.uint16)      # all scores equal
    v = np.zeros((pages * P, D), dtype=np.float32)
    for pos in range(L + n):
        v[pos, pos] = 1.0                                      # V_pos = e_pos
    v_cache = W.f32_to_bf16_bits(v).reshape(pages, P, 1, D).transpose(0, 2, 1, 3).copy()
    q = W.f32_to_bf16_bits(np.ones((n, 1, D), dtype=np.float32))
    out, lse = oracle.verify_attn(q, k_cache, v_cache, np.arange(pages, dtype=np.int32)[None], np.array([L], np.int32),
                                  np.array([0, n], np.int32), parent, 1.0)
    for i, vis in enumerate(gold["visible"]):
        want = np.zeros(D)
        keys = list(range(L)) + [L + j for j in vis]
        want[keys] = 1.0 / len(keys)
        np.testing.assert_allclose(out[i, 0], want, atol=1e-15)
        np.testing.assert_allclose(lse[i, 0], np.log(len(keys)), atol=1e-15)
    # siblings never see each other
    assert out[2, 0, L + 1] == 0.0 and out[1, 0, L + 2] == 0.0


def test_softmax_invariants():
    wl = _small([("tree", 8, 3), ("chain", 3)], [40, 9], hq=4, hkv=2)
    out, lse = _run(wl)
    sp = wl.spec
    for b in range(2):
        lo, hi = int(wl.node_offsets[b]), int(wl.node_offsets[b + 1])
        n, L = hi - lo, int(wl.ctx_lens[b])
        mask = _dense_mask(wl.tree_parent[lo:hi])
        for hq in range(4):
            K = _gather_kv(wl.k_cache, wl.block_table, b, hq // 2, L + n, 16)
            V = _gather_kv(wl.v_cache, wl.block_table, b, hq // 2, L + n, 16)
            for i in range(n):
                vis = np.concatenate([np.ones(L, bool), mask[i]])
                s = wl.sm_scale * (K[vis] @ _f64(wl.q[lo + i, hq]))
                l = lse[lo + i, hq]
                assert abs(np.exp(s - l).sum() - 1.0) < 1e-12            # probabilities sum to one
                assert s.max() <= l <= s.max() + np.log(vis.sum()) + 1e-12  # lse bounds
                o = out[lo + i, hq]
                assert np.all(o <= V[vis].max(axis=0) + 1e-12) and np.all(o >= V[vis].min(axis=0) - 1e-12)


def test_constant_v_gives_constant_output():
    wl = _small([("tree", 6, 3)], [30])
    wl.v_cache[...] = W.f32_to_bf16_bits(np.array([0.75], dtype=np.float32))[0]
    out, _ = _run(wl)
    np.testing.assert_allclose(out, 0.75, atol=1e-14)


def test_page_permutation_invariance():
    wl = _small([("tree", 8, 3), ("chain", 5)], [70, 33], shuffle=False)
    out, lse = _run(wl)
    rng = np.random.default_rng(0)
    perm = rng.permutation(wl.num_pages)            # new physical page of old page p is perm[p]
    k2 = np.empty_like(wl.k_cache); v2 = np.empty_like(wl.v_cache)
    k2[perm] = wl.k_cache; v2[perm] = wl.v_cache
    bt2 = perm[wl.block_table].astype(np.int32)
    out2, lse2 = oracle.verify_attn(wl.q, k2, v2, bt2, wl.ctx_lens, wl.node_offsets, wl.tree_parent, wl.sm_scale)
    np.testing.assert_array_equal(out, out2)
    np.testing.assert_array_equal(lse, lse2)


def test_unused_slots_are_never_read():
    """Cache slots past L+n (tail of the last page) may hold anything, even NaN."""
    wl = _small([("tree", 5, 2)], [22], shuffle=False)       # 27 positions, 2 pages, 5 unused slots
    out, lse = _run(wl)
    wl.k_cache[1, :, 11:, :] = 0x7FC0
    wl.v_cache[1, :, 11:, :] = 0x7FC0
    out2, lse2 = _run(wl)
    np.testing.assert_array_equal(out, out2)
    np.testing.assert_array_equal(lse, lse2)


def test_sibling_order_permutation_permutes_outputs():
    parent = np.array([-1, 0, 0, 1, 2], dtype=np.int32)
    wl = _small([("chain", 5)], [21], shuffle=False)
    wl.tree_parent[:] = parent
    out, lse = _run(wl)
    # swap nodes 1<->2 and their children 3<->4: q rows and cache slots move with the nodes
    sw = np.array([0, 2, 1, 4, 3])
    wl2 = _small([("chain", 5)], [21], shuffle=False)
    wl2.tree_parent[:] = parent            # the relabelled tree has the same parent array
    wl2.q[:] = wl.q[sw]
    L = 21
    for cache, src in ((wl2.k_cache, wl.k_cache), (wl2.v_cache, wl.v_cache)):
        flat = cache.transpose(0, 2, 1, 3).reshape(-1, cache.shape[1], 128).copy()
        sflat = src.transpose(0, 2, 1, 3).reshape(-1, src.shape[1], 128)
        flat[L:L + 5] = sflat[L + sw]
        cache[...] = flat.reshape(cache.shape[0], 16, cache.shape[1], 128).transpose(0, 2, 1, 3)
    out2, lse2 = _run(wl2)
    np.testing.assert_allclose(out2, out[sw], atol=1e-13)
    np.testing.assert_allclose(lse2, lse[sw], atol=1e-13)


def test_split_merge_identity():
    """Merging per-chunk (o, lse) partials by their log-sum-exp reproduces the whole, for any split."""
    wl = _small([("chain", 1)], [95], hq=2, hkv=1, shuffle=False)
    out, lse = _run(wl)
    K = _gather_kv(wl.k_cache, wl.block_table, 0, 0, 96, 16)
    V = _gather_kv(wl.v_cache, wl.block_table, 0, 0, 96, 16)
    q = _f64(wl.q[0, 1])
    s = wl.sm_scale * (K @ q)
    cuts = [0, 7, 40, 41, 96]
    parts = []
    for a, b in zip(cuts[:-1], cuts[1:]):
        l = np.log(np.exp(s[a:b]).sum())
        parts.append((np.exp(s[a:b] - l) @ V[a:b], l))
    tot = np.log(sum(np.exp(l) for _, l in parts))
    merged = sum(np.exp(l - tot) * o for o, l in parts)
    np.testing.assert_allclose(tot, lse[0, 1], atol=1e-12)
    np.testing.assert_allclose(merged, out[0, 1], atol=1e-12)


def test_rejects_malformed_tree():
    wl = _small([("chain", 4)], [10])
    wl.tree_parent[2] = 3
    with pytest.raises(ValueError):
        _run(wl)

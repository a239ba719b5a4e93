"""Pins of the oracle functions for the steps around the verify pass (CPU only): Prepare(d) with its
[SPEC] leaves and position ids, the [SPEC] leaf of an accepted path, and the commit of the accepted
tokens to the paged cache.  Each is checked against what the paper fixes (its worked example), against
hand-worked cases, against an independent formulation, and inside a multi-step lossless loop."""
import json
import os

import numpy as np
import pytest

import oracle
from paper_2510_07535_b200 import workloads as W


def _golden(golden_dir, name):
    with open(os.path.join(golden_dir, name)) as f:
        return json.load(f)


# ----------------------------------------------------------------------------- Prepare(d), [SPEC] leaf

def test_prepare_matches_the_papers_example(golden_dir):
    g = _golden(golden_dir, "spec_prepare_example.json")
    i32 = lambda a: np.asarray(a, np.int32)
    offs, par, drf, ids, pos = oracle.prepare_spec_tree(i32(g["in"]["node_offsets"]), i32(g["in"]["tree_parent"]),
                                                        i32(g["in"]["draft_tokens"]), i32([g["ctx_len"]]), g["spec_token"])
    assert offs.tolist() == g["out"]["node_offsets"]
    assert par.tolist() == g["out"]["tree_parent"]
    assert drf.tolist() == g["out"]["draft_tokens"]
    assert ids.tolist() == g["out"]["input_ids"]
    assert pos.tolist() == g["out"]["position_ids"]
    # the same parents as the mask example of the Decode-Stage paragraph: the attention pins apply to prepared trees
    assert par.tolist() == _golden(golden_dir, "decode_stage_mask_example.json")["tree_parent"]
    for case in g["accepted"]:
        path = np.full((1, 8), -1, np.int32)
        path[0, :len(case["path"])] = case["path"]
        leaf = oracle.spec_leaf(offs, par, drf, i32([len(case["path"])]), path)
        assert leaf.tolist() == [case["spec_node"]]


def test_prepare_invariants_on_random_trees():
    rng = np.random.default_rng(3)
    for trial in range(50):
        B = int(rng.integers(1, 5))
        parents = [W.random_tree_parents(rng, int(rng.integers(1, 33)), 8) for _ in range(B)]
        counts = np.array([len(p) for p in parents])
        offs_in = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
        par_in = np.concatenate(parents).astype(np.int32)
        tok_in = rng.integers(0, 5000, size=len(par_in)).astype(np.int32)
        ctx = rng.integers(0, 100000, size=B).astype(np.int32)
        offs, par, drf, ids, pos = oracle.prepare_spec_tree(offs_in, par_in, tok_in, ctx, 7777)
        assert np.array_equal(offs, 2 * offs_in)                      # "the same number of [SPEC] as tree nodes"
        for b in range(B):
            n, o = int(counts[b]), int(offs[b])
            p = par[o:o + 2 * n]
            assert p[0] == -1 and np.all(p[1:] < np.arange(1, 2 * n)) and np.all(p[1:] >= 0)   # still a valid order
            assert np.array_equal(p[:n], parents[b])                  # the drafted tree is unchanged
            assert np.array_equal(p[n:], np.arange(n))                # leaf j follows the path that ends in node j
            assert np.array_equal(drf[o:o + n], tok_in[offs_in[b]:offs_in[b + 1]]) and np.all(drf[o + n:o + 2 * n] == -1)
            assert np.array_equal(ids[o:o + n], drf[o:o + n]) and np.all(ids[o + n:o + 2 * n] == 7777)
            depth = W.tree_depths(p)                                  # independent recursion d[i] = d[parent] + 1
            assert np.array_equal(pos[o:o + 2 * n], ctx[b] + depth)
            assert np.array_equal(depth[n:], depth[:n] + 1)           # a [SPEC] sits right after its path
            # no drafted node has a [SPEC] as parent: leaves stay leaves
            assert np.all(p < n)


def test_spec_leaf_of_prepared_and_unprepared_trees():
    rng = np.random.default_rng(4)
    par = W.random_tree_parents(rng, 20, 6)
    tok = rng.integers(0, 100, size=20).astype(np.int32)
    offs, p2, d2, _, _ = oracle.prepare_spec_tree(np.array([0, 20], np.int32), par, tok, np.array([5], np.int32), 1)
    for last in range(20):
        chain = [last]
        while par[chain[-1]] >= 0:
            chain.append(int(par[chain[-1]]))
        chain = chain[::-1]
        path = np.full((1, 64), -1, np.int32)
        path[0, :len(chain)] = chain
        assert oracle.spec_leaf(offs, p2, d2, np.array([len(chain)], np.int32), path).tolist() == [20 + last]
        # the tree as drafted has no [SPEC] at all
        assert oracle.spec_leaf(np.array([0, 20], np.int32), par, np.abs(tok), np.array([len(chain)], np.int32), path).tolist() == [-1]
    # two [SPEC]-like children of the same node: the lowest index; a [SPEC] under another node does not count
    parents = np.array([-1, 0, 0, 1, 1, 0], np.int32)
    tokens = np.array([3, 4, -1, -1, -1, -1], np.int32)
    path = np.array([[0, 1, -1, -1]], np.int32)
    assert oracle.spec_leaf(np.array([0, 6], np.int32), parents, tokens, np.array([2], np.int32), path).tolist() == [3]
    assert oracle.spec_leaf(np.array([0, 6], np.int32), parents, tokens, np.array([1], np.int32), path).tolist() == [2]


def test_acceptance_never_walks_into_spec_leaves_of_a_prepared_tree():
    """[SPEC] leaves double the tree but change nothing of the acceptance (they are never candidates)."""
    rng = np.random.default_rng(8)
    for trial in range(100):
        n = int(rng.integers(1, 33))
        par = W.random_tree_parents(rng, n, 8)
        tok = rng.integers(0, 6, size=n).astype(np.int32)
        am = rng.integers(0, 6, size=n).astype(np.int32)
        offs = np.array([0, n], np.int32)
        alen, path, bonus = oracle.accept_from_argmax(offs, par, tok, am)
        o2, p2, d2, _, _ = oracle.prepare_spec_tree(offs, par, tok, np.array([9], np.int32), 5)
        am2 = np.concatenate([am, rng.integers(0, 6, size=n).astype(np.int32)])   # rows of the [SPEC] leaves: anything
        alen2, path2, bonus2 = oracle.accept_from_argmax(o2, p2, d2, am2)
        assert np.array_equal(alen, alen2) and np.array_equal(path, path2) and np.array_equal(bonus, bonus2)


# ----------------------------------------------------------------------------- commit of the accepted tokens

def _numbered_cache(num_pages, hkv, page, seed):
    """Every element distinct enough to tell slots, heads and K from V apart."""
    rng = np.random.default_rng(seed)
    return (rng.integers(0, 2 ** 16, size=(num_pages, hkv, page, W.HEAD_DIM), dtype=np.uint16),
            rng.integers(0, 2 ** 16, size=(num_pages, hkv, page, W.HEAD_DIM), dtype=np.uint16))


def _logical(cache, table_row, page, positions):
    positions = np.asarray(positions)
    return cache[table_row[positions // page], :, positions % page, :]


def test_commit_hand_worked_cases(golden_dir):
    g = _golden(golden_dir, "kv_commit_cases.json")
    P = g["page_size"]
    for case in g["cases"]:
        bt = np.asarray(case["block_table"], np.int32)
        k0, v0 = _numbered_cache(int(bt.max()) + 1, 2, P, 11)
        k, v = k0.copy(), v0.copy()
        ctx = np.asarray(case["ctx_lens"], np.int32).copy()
        path = np.asarray(case["accept_path"], np.int32)
        oracle.kv_commit(k, v, bt, ctx, np.asarray(case["node_offsets"], np.int32), np.asarray(case["accept_len"], np.int32), path)
        assert ctx.tolist() == case["new_ctx_lens"], case["name"]
        touched = np.zeros(k.shape[:3], bool)
        for a in case["after"]:
            b, pos, src = a["b"], a["pos"], a["from"]
            for cache, orig in ((k, k0), (v, v0)):
                got = cache[bt[b, pos // P], :, pos % P, :]
                want = orig[bt[b, src // P], :, src % P, :]
                assert np.array_equal(got, want), (case["name"], a)
            touched[bt[b, pos // P], :, pos % P] = True
        assert np.array_equal(k[~touched], k0[~touched]) and np.array_equal(v[~touched], v0[~touched]), case["name"]


def test_commit_equals_fancy_indexing_on_the_logical_view():
    """Independent formulation: gather each sequence's logical token rows through the block table, apply
    text[L + k] = text[L + path[k]] as one numpy fancy-index assignment (right-hand side evaluated first),
    scatter back."""
    rng = np.random.default_rng(21)
    for trial in range(30):
        B, hkv, page = int(rng.integers(1, 5)), int(rng.integers(1, 4)), int(rng.choice([4, 16, 32]))
        parents = [W.random_tree_parents(rng, int(rng.integers(1, 41)), 8) for _ in range(B)]
        counts = np.array([len(p) for p in parents])
        offs = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
        ctx = rng.integers(0, 70, size=B).astype(np.int32)
        pages_per = (ctx + counts + page - 1) // page
        maxp = int(pages_per.max()) + 1
        table = rng.permutation(B * maxp).astype(np.int32).reshape(B, maxp)
        k0, v0 = _numbered_cache(B * maxp, hkv, page, 100 + trial)
        alen = np.zeros(B, np.int32)
        path = np.full((B, 64), -1, np.int32)
        for b in range(B):                       # a random root path of each tree
            last = int(rng.integers(0, counts[b]))
            chain = [last]
            while parents[b][chain[-1]] >= 0:
                chain.append(int(parents[b][chain[-1]]))
            chain = chain[::-1]
            alen[b] = len(chain)
            path[b, :len(chain)] = chain
        k, v, c = k0.copy(), v0.copy(), ctx.copy()
        oracle.kv_commit(k, v, table, c, offs, alen, path)
        assert np.array_equal(c, ctx + alen)
        ke, ve = k0.copy(), v0.copy()
        for b in range(B):
            L, a = int(ctx[b]), int(alen[b])
            span = np.arange(L + counts[b])
            for cache in (ke, ve):
                text = _logical(cache, table[b], page, span).copy()      # [positions, hkv, D]
                text[L + np.arange(a)] = text[L + path[b, :a]]
                cache[table[b][span // page], :, span % page, :] = text
        assert np.array_equal(k, ke) and np.array_equal(v, ve)


def test_commit_rejects_paths_that_are_not_root_paths_in_order():
    bt = np.arange(4, dtype=np.int32).reshape(1, 4)
    k, v = _numbered_cache(4, 1, 4, 1)
    offs = np.array([0, 6], np.int32)
    for alen, p in ((0, [0, 1, 2]), (2, [1, 2, -1]), (3, [0, 2, 2]), (3, [0, 3, 2]), (2, [0, 6, -1]), (7, [0, 1, 2])):
        with pytest.raises(ValueError):
            oracle.kv_commit(k.copy(), v.copy(), bt, np.array([3], np.int32), offs, np.array([alen], np.int32),
                             np.array([p + [-1] * (8 - len(p))], np.int32))


# ----------------------------------------------------------------------------- the whole loop, 200 steps

def test_lossless_loop_with_spec_leaves_and_commits():
    """Algorithm 1 on a toy model, 200 verification steps, every step with the oracle's Prepare / accept /
    [SPEC] pick / commit: the committed text equals plain one-token-at-a-time iteration of the toy model
    ("lossless"), the cache holds exactly the rows of that text at their positions, and the [SPEC] leaf
    picked is the one whose position id is the first uncommitted position."""
    toy = W.ToyLoop(batch=3, seed=17)
    k, v = toy.initial_cache()
    ctx = toy.ctx0.copy()
    roots = [int(toy.text(b, int(ctx[b]) + 1)[-1]) for b in range(toy.B)]
    emitted = [[] for _ in range(toy.B)]
    total_accepted = 0
    for step in range(200):
        kinds, offs, par, tok = toy.draft(roots)
        # chains are verified as drafted, trees with one [SPEC] leaf per node (the hybrid of Section 3.2.3);
        # Prepare runs on the whole batch and the chains keep their own halves
        o2, p2, d2, ids2, pos2 = oracle.prepare_spec_tree(offs, par, tok, ctx, toy.spec_token)
        seq_par, seq_tok, seq_ids, seq_pos = [], [], [], []
        for b in range(toy.B):
            n = int(offs[b + 1] - offs[b])
            take = n if kinds[b] == "chain" else 2 * n
            sl = slice(int(o2[b]), int(o2[b]) + take)
            seq_par.append(p2[sl]); seq_tok.append(d2[sl]); seq_ids.append(ids2[sl]); seq_pos.append(pos2[sl])
        v_offs = np.concatenate([[0], np.cumsum([len(x) for x in seq_par])]).astype(np.int32)
        v_par, v_tok, v_ids = np.concatenate(seq_par), np.concatenate(seq_tok), np.concatenate(seq_ids)
        for b in range(toy.B):                                     # the verifier's K/V of the drafted nodes
            n = len(seq_par[b])
            toy.write_rows(k, v, b, int(ctx[b]) + np.arange(n), seq_ids[b], seq_pos[b])
        alen, path, bonus, _ = oracle.tree_accept(toy.logits(v_ids), v_tok, v_offs, v_par, 64)
        leaf = oracle.spec_leaf(v_offs, v_par, v_tok, alen, path)
        old_ctx = ctx.copy()
        oracle.kv_commit(k, v, toy.block_table, ctx, v_offs, alen, path)
        for b in range(toy.B):
            a = int(alen[b])
            assert 1 <= a <= 9                                     # the paper's bounds: at least the root, at most depth + 1
            emitted[b].extend(int(seq_ids[b][j]) for j in path[b, :a])
            assert ctx[b] == old_ctx[b] + a
            if kinds[b] == "tree":
                assert leaf[b] >= 0 and seq_pos[b][leaf[b]] == ctx[b]      # the [SPEC] right after the accepted path
            else:
                assert leaf[b] == -1
            roots[b] = int(bonus[b])
            total_accepted += a
    assert total_accepted > 200 * toy.B * 1.5                      # drafts do get accepted
    for b in range(toy.B):
        L = int(ctx[b])
        text = toy.text(b, L + 1)
        assert emitted[b] == text[int(toy.ctx0[b]):L].tolist()     # lossless
        assert roots[b] == text[L]
        pos = np.arange(L)
        assert np.array_equal(toy.read_rows(k, b, pos), toy.kv_rows(text[:L], pos, toy.Hkv, 0))
        assert np.array_equal(toy.read_rows(v, b, pos), toy.kv_rows(text[:L], pos, toy.Hkv, 1))


def _commit_case_holds(commit, case, P):
    """True iff `commit` (same signature as oracle.kv_commit) reproduces a hand-worked case."""
    bt = np.asarray(case["block_table"], np.int32)
    k0, v0 = _numbered_cache(int(bt.max()) + 1, 2, P, 11)
    k, v = k0.copy(), v0.copy()
    ctx = np.asarray(case["ctx_lens"], np.int32).copy()
    commit(k, v, bt, ctx, np.asarray(case["node_offsets"], np.int32), np.asarray(case["accept_len"], np.int32),
           np.asarray(case["accept_path"], np.int32))
    ok = ctx.tolist() == case["new_ctx_lens"]
    for a in case["after"]:
        b, pos, src = a["b"], a["pos"], a["from"]
        for cache, orig in ((k, k0), (v, v0)):
            ok = ok and np.array_equal(cache[bt[b, pos // P], :, pos % P, :], orig[bt[b, src // P], :, src % P, :])
    return ok


@pytest.mark.parametrize("mistake", ["backwards_in_place", "swapped_heads", "no_length_update", "k_only"])
def test_planted_commit_mistakes_fail_the_hand_worked_cases(golden_dir, mistake):
    """Plausible slips, written out as wrong commits on the CPU, are each rejected by the hand-worked cases (which
    the oracle's commit reproduces)."""
    g = _golden(golden_dir, "kv_commit_cases.json")
    P = g["page_size"]

    def wrong(k, v, bt, ctx, offs, alen, path):
        for b in range(len(ctx)):
            L, a = int(ctx[b]), int(alen[b])
            ks = range(a - 1, -1, -1) if mistake == "backwards_in_place" else range(a)
            for cache in ((k,) if mistake == "k_only" else (k, v)):
                rows = {kk: cache[bt[b, (L + path[b, kk]) // P], :, (L + path[b, kk]) % P, :].copy() for kk in range(a)}
                for kk in ks:
                    row = rows[kk]
                    if mistake == "backwards_in_place":      # re-reads sources that were already overwritten
                        row = cache[bt[b, (L + path[b, kk]) // P], :, (L + path[b, kk]) % P, :].copy()
                    if mistake == "swapped_heads":
                        row = row[::-1]
                    cache[bt[b, (L + kk) // P], :, (L + kk) % P, :] = row
            if mistake != "no_length_update":
                ctx[b] = L + a

    assert all(_commit_case_holds(oracle.kv_commit, c, P) for c in g["cases"])
    assert not all(_commit_case_holds(wrong, c, P) for c in g["cases"])

"""Pins for the acceptance oracle (CPU only): hand-worked cases, bounds the paper states,
losslessness on a toy model, and a closed-form expectation."""
import json
import os

import numpy as np
import pytest

import oracle
from paper_2510_07535_b200 import workloads as W


def _logits_with_argmax(am, vocab, rng):
    """fp32 rows whose unique maximum sits at am[i]."""
    lg = rng.standard_normal((len(am), vocab)).astype(np.float32)
    lg[np.arange(len(am)), am] = 50.0
    return lg


def test_hand_worked_cases(golden_dir):
    with open(os.path.join(golden_dir, "acceptance_cases.json")) as f:
        gold = json.load(f)
    rng = np.random.default_rng(1)
    for case in gold["cases"]:
        am = np.array(case["argmax"], dtype=np.int32)
        lg = _logits_with_argmax(am, 16, rng)
        alen, path, bonus, am_out = oracle.tree_accept(lg, np.array(case["draft_tokens"], np.int32),
                                                       np.array(case["node_offsets"], np.int32),
                                                       np.array(case["tree_parent"], np.int32), path_stride=8)
        assert am_out.tolist() == case["argmax"], case["name"]
        assert alen.tolist() == case["accept_len"], case["name"]
        assert bonus.tolist() == case["bonus_token"], case["name"]
        for b, p in enumerate(case["accept_path"]):
            assert path[b, :len(p)].tolist() == p, case["name"]
            assert np.all(path[b, len(p):] == -1), case["name"]


def test_tie_takes_lowest_index(golden_dir):
    with open(os.path.join(golden_dir, "acceptance_cases.json")) as f:
        t = json.load(f)["tie_case"]
    lg = np.zeros((3, t["vocab"]), dtype=np.float32)
    for r, pos in enumerate(t["row_max_positions"]):
        lg[r, pos] = 2.5
    alen, path, bonus, am = oracle.tree_accept(lg, np.array(t["draft_tokens"], np.int32),
                                               np.array(t["node_offsets"], np.int32),
                                               np.array(t["tree_parent"], np.int32), path_stride=4)
    assert am[0] == 4
    assert alen.tolist() == t["accept_len"] and bonus.tolist() == t["bonus_token"]
    assert path[0, :2].tolist() == t["accept_path"][0]


def test_argmax_matches_numpy_and_edge_values():
    rng = np.random.default_rng(2)
    lg = rng.standard_normal((7, 1001)).astype(np.float32)
    lg[1, 17] = lg[1, 900] = 9.0                       # tie -> 17
    lg[2, :] = -np.inf                                 # all -inf -> 0
    lg[3, :] = 0.0; lg[3, 5] = -0.0                    # +0 == -0 -> 0
    lg[4, 3] = np.nan; lg[4, 10] = 30.0                # NaN never wins
    lg[5, :] = np.nan                                  # all NaN -> 0
    lg[6, -1] = 99.0                                   # last element
    am = oracle.row_argmax(lg)
    assert am[0] == int(np.argmax(lg[0]))              # numpy argmax also returns the first maximum
    assert am.tolist()[1:] == [17, 0, 0, 10, 0, 1000]


def test_length_bounds_on_random_trees():
    """1 <= accept_len <= max depth + 1 (a step always emits the root; depth 8 gives at most 9)."""
    rng = np.random.default_rng(3)
    for trial in range(200):
        md = int(rng.integers(1, 9))
        n = int(rng.integers(1, min(64, 1 + 2 * md) + 1))
        par = W.random_tree_parents(rng, n, md)
        depth = W.tree_depths(par)
        tok = rng.integers(0, 6, size=n).astype(np.int32)
        am = rng.integers(0, 6, size=n).astype(np.int32)
        alen, path, bonus = oracle.accept_from_argmax(np.array([0, n], np.int32), par, tok, am)
        assert 1 <= alen[0] <= depth.max() + 1 <= 9
        p = path[0, :alen[0]]
        assert p[0] == 0 and np.all(path[0, alen[0]:] == -1)
        for a, c in zip(p[:-1], p[1:]):               # a valid root path whose tokens match
            assert par[c] == a and tok[c] == am[a]
        assert bonus[0] == am[p[-1]]
        # maximality: no accepted node is deeper
        ok = np.zeros(n, bool); ok[0] = True
        for i in range(1, n):
            ok[i] = ok[par[i]] and tok[i] == am[par[i]]
        assert depth[ok].max() + 1 == alen[0]
        assert p[-1] == np.flatnonzero(ok & (depth == depth[ok].max()))[0]


def test_lossless_on_toy_model():
    """Verify-accept-commit over random trees emits exactly what one-token-at-a-time greedy decoding emits."""
    V = 97
    f = lambda t: (t * 31 + 7) % V                     # toy "target model": next token is f(last token)
    rng = np.random.default_rng(4)
    plain = [5]
    for _ in range(400):
        plain.append(f(plain[-1]))
    emitted = [5]
    root = 5
    while len(emitted) < 300:
        md = int(rng.integers(1, 9))
        n = int(rng.integers(1, min(32, 1 + 2 * md) + 1))
        par = W.random_tree_parents(rng, n, md)
        tok = np.zeros(n, dtype=np.int32)
        tok[0] = root
        for i in range(1, n):                          # drafter: right with probability 0.6
            tok[i] = f(tok[par[i]]) if rng.random() < 0.6 else int(rng.integers(0, V))
        lg = _logits_with_argmax(np.array([f(int(t)) for t in tok]), V, rng)
        alen, path, bonus, _ = oracle.tree_accept(lg, tok, np.array([0, n], np.int32), par)
        acc = [int(tok[j]) for j in path[0, :alen[0]]]
        assert acc[0] == root
        emitted.extend(acc[1:])
        emitted.append(int(bonus[0]))
        root = int(bonus[0])
    assert emitted == plain[:len(emitted)]


def _truncated_geometric_variance(n, p):
    k = np.arange(1, n + 1)
    pk = np.array([p ** (j - 1) * (1 - p) for j in range(1, n)] + [p ** (n - 1)])
    assert abs(pk.sum() - 1) < 1e-12
    return float((pk * k * k).sum() - (pk * k).sum() ** 2)


def test_chain_acceptance_closed_form():
    """Chain of n nodes with each edge planted w.p. p: E[accept_len] = (1 - p^n) / (1 - p)."""
    n, p, trials, V = 8, 0.7, 10000, 512
    rng = np.random.default_rng(5)
    par = W.chain_parents(n)
    offs = np.arange(0, (trials + 1) * n, n, dtype=np.int32)
    tok = rng.integers(0, V, size=trials * n).astype(np.int32)
    am = rng.integers(0, V, size=trials * n).astype(np.int32)
    hit = rng.random(trials * n) < p
    idx = np.arange(trials * n)
    child = idx[idx % n != 0]
    # planted edge: the parent's arg-max is the child's token; unplanted: force a mismatch
    am[child - 1] = np.where(hit[child], tok[child], (tok[child] + 1) % V)
    alen, _, _ = oracle.accept_from_argmax(offs, np.tile(par, trials), tok, am)
    mean = alen.mean()
    expect = (1 - p ** n) / (1 - p)
    # P(len = k) = p^(k-1) (1 - p) for k < n and p^(n-1) for k = n: variance 4.858 at n = 8, p = 0.7;
    # the bound is 4 sigma of the mean of `trials` draws (0.088)
    assert abs(mean - expect) < 4 * np.sqrt(_truncated_geometric_variance(n, p) / trials), (mean, expect)
    assert abs(expect - 3.1412) < 1e-3


def test_planted_logits_generator_agrees_with_closed_form():
    """The workload generator's planting (+10 on the parent's row) drives acceptance as designed."""
    B = 1024
    spec = W.Spec("p8", 4, 1, [16] * B, [("chain", 8)] * B, plant_prob=0.7, vocab=4096, seed=11)
    wl = W.generate(spec, threads=1)
    alen, _, _, _ = oracle.tree_accept(wl.logits, wl.draft_tokens, wl.node_offsets, wl.tree_parent)
    # 4 sigma of the mean of 1024 chains (0.28); an unplanted edge matches with probability ~ 1/4096 only
    assert abs(alen.mean() - 3.1412) < 4 * np.sqrt(_truncated_geometric_variance(8, 0.7) / B), alen.mean()
    assert alen.min() >= 1 and alen.max() <= 8


def test_rejects_bad_tree():
    with pytest.raises(ValueError):
        oracle.accept_from_argmax(np.array([0, 3], np.int32), np.array([-1, 2, 0], np.int32),
                                  np.zeros(3, np.int32), np.zeros(3, np.int32))

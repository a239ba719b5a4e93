"""The steps around the verify pass on the GPU, through the C ABI, against the CPU oracle: Prepare(d) with its
[SPEC] leaves, the [SPEC] leaf of the accepted path, the commit of accepted tokens to the paged cache - each bit
for bit - and Algorithm 1's loop run for 200 verification steps with cache, lengths and acceptance results
staying on the device."""
import json
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2510_07535_b200 import OwlContext, make_dims, owl_howl_route, workloads as W

pytestmark = pytest.mark.gpu

DEV = "cuda"


def dev_i32(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(DEV)


def dev_bf16(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(DEV).view(torch.bfloat16)


def bits_of(t):
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


def random_drafts(rng, B, max_n):
    parents = [W.random_tree_parents(rng, int(rng.integers(1, max_n + 1)), 8) for _ in range(B)]
    counts = np.array([len(p) for p in parents])
    offs = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
    return parents, counts, offs, np.concatenate(parents).astype(np.int32)


def gpu_prepare(ctx, offs, par, tok, ctx_lens, spec_token, uniform=False):
    B, N = len(offs) - 1, len(par)
    d = make_dims(batch=B, total_nodes=N, max_nodes=int(np.diff(offs).max()))
    outs = [torch.full((B + 1,), -7, dtype=torch.int32, device=DEV)] + [torch.full((2 * N,), -7, dtype=torch.int32, device=DEV) for _ in range(4)]
    ctx.owl_prepare_spec_tree(d, None if uniform else dev_i32(offs), dev_i32(par), dev_i32(tok), dev_i32(ctx_lens), spec_token, *outs)
    return outs


def test_prepare_matches_oracle_and_the_papers_example(golden_dir):
    ctx = OwlContext(make_dims(batch=8, total_nodes=8 * 32, max_nodes=32))
    g = json.load(open(os.path.join(golden_dir, "spec_prepare_example.json")))
    outs = gpu_prepare(ctx, np.array(g["in"]["node_offsets"]), np.array(g["in"]["tree_parent"]), np.array(g["in"]["draft_tokens"]),
                       np.array([g["ctx_len"]]), g["spec_token"])
    assert ctx.owl_get_status() == 0
    for got, key in zip(outs, ("node_offsets", "tree_parent", "draft_tokens", "input_ids", "position_ids")):
        assert got.cpu().tolist() == g["out"][key], key
    rng = np.random.default_rng(31)
    for trial in range(20):
        B = int(rng.integers(1, 9))
        _, counts, offs, par = random_drafts(rng, B, 32)
        tok = rng.integers(0, 128256, size=len(par)).astype(np.int32)
        lens = rng.integers(0, 131072, size=B).astype(np.int32)
        outs = gpu_prepare(ctx, offs, par, tok, lens, 128255)
        assert ctx.owl_get_status() == 0
        for got, ref in zip(outs, oracle.prepare_spec_tree(offs, par, tok, lens, 128255)):
            np.testing.assert_array_equal(got.cpu().numpy(), ref)
    # uniform batches may pass NULL offsets
    par = np.tile(W.random_tree_parents(rng, 9, 4), 3).astype(np.int32)
    offs = np.array([0, 9, 18, 27], np.int32)
    tok = rng.integers(0, 99, size=27).astype(np.int32)
    outs = gpu_prepare(ctx, offs, par, tok, np.array([5, 6, 7]), 3, uniform=True)
    for got, ref in zip(outs, oracle.prepare_spec_tree(offs, par, tok, np.array([5, 6, 7], np.int32), 3)):
        np.testing.assert_array_equal(got.cpu().numpy(), ref)
    ctx.close()


def test_prepare_errors():
    ctx = OwlContext(make_dims(batch=2, total_nodes=66, max_nodes=33))
    one = torch.zeros(80, dtype=torch.int32, device=DEV)
    # 33 drafted nodes would make a 66-node tree: refused on the host, nothing launched
    n0 = ctx.launch_count()
    d = make_dims(batch=1, total_nodes=33, max_nodes=33)
    assert ctx.owl_prepare_spec_tree(d, None, one, one, one, 1, one, one, one, one, one, check=False) == -2
    d = make_dims(batch=1, total_nodes=4, max_nodes=4)
    assert ctx.owl_prepare_spec_tree(d, None, None, one, one, 1, one, one, one, one, one, check=False) == -1
    assert ctx.launch_count() == n0
    # a malformed tree in sequence 1: reported, its rows unwritten, sequence 0 prepared
    offs, par = np.array([0, 3, 6], np.int32), np.array([-1, 0, 0, -1, 2, 0], np.int32)
    tok = np.arange(6, dtype=np.int32)
    outs = gpu_prepare(ctx, offs, par, tok, np.array([10, 20]), 9)
    assert ctx.owl_get_status() == -4
    ref = oracle.prepare_spec_tree(np.array([0, 3], np.int32), par[:3], tok[:3], np.array([10], np.int32), 9)
    for got, r in zip(outs[1:], ref[1:]):
        assert got.cpu().tolist()[:6] == r.tolist() and got.cpu().tolist()[6:] == [-7] * 6
    ctx.close()


def test_spec_leaf_output_matches_oracle():
    rng = np.random.default_rng(41)
    V = 20000
    ctx = OwlContext(make_dims(batch=6, total_nodes=6 * 64, max_nodes=64, vocab=V))
    for trial in range(6):
        B = int(rng.integers(1, 7))
        _, counts, offs, par = random_drafts(rng, B, 32)
        tok = rng.integers(0, V, size=len(par)).astype(np.int32)
        o2, p2, d2, _, _ = oracle.prepare_spec_tree(offs, par, tok, np.zeros(B, np.int32), V - 1)
        if trial % 2:                      # odd trials: trees as drafted, no [SPEC] anywhere
            o2, p2, d2 = offs, par, tok
        N = len(p2)
        lg = rng.standard_normal((N, V)).astype(np.float32)
        for i in range(N):                 # make most edges match so that paths get long
            b = int(np.searchsorted(o2, i, side="right") - 1)
            if p2[i] >= 0 and d2[i] >= 0 and rng.random() < 0.8:
                lg[o2[b] + p2[i], d2[i]] += 12
        d = make_dims(batch=B, total_nodes=N, max_nodes=int(np.diff(o2).max()), vocab=V)
        alen = torch.zeros(B, dtype=torch.int32, device=DEV); path = torch.zeros((B, 64), dtype=torch.int32, device=DEV)
        bonus = torch.zeros(B, dtype=torch.int32, device=DEV); leaf = torch.full((B,), -9, dtype=torch.int32, device=DEV)
        ctx.owl_tree_accept_spec(d, torch.from_numpy(lg).to(DEV), dev_i32(d2), dev_i32(o2), dev_i32(p2), alen, path, bonus, leaf)
        assert ctx.owl_get_status() == 0
        r_alen, r_path, r_bonus, _ = oracle.tree_accept(lg, d2, o2, p2, 64)
        np.testing.assert_array_equal(alen.cpu().numpy(), r_alen)
        np.testing.assert_array_equal(path.cpu().numpy(), r_path)
        np.testing.assert_array_equal(bonus.cpu().numpy(), r_bonus)
        np.testing.assert_array_equal(leaf.cpu().numpy(), oracle.spec_leaf(o2, p2, d2, r_alen, r_path))
        assert r_alen.max() > 1
    ctx.close()


def _commit_case(rng, B, hkv, page):
    parents, counts, offs, par = random_drafts(rng, B, 64)
    lens = rng.integers(0, 200, size=B).astype(np.int32)
    maxp = int(((lens + counts + page - 1) // page).max()) + 1
    table = rng.permutation(B * maxp).astype(np.int32).reshape(B, maxp)
    k = rng.integers(0, 2 ** 16, size=(B * maxp, hkv, page, 128), dtype=np.uint16)
    v = rng.integers(0, 2 ** 16, size=(B * maxp, hkv, page, 128), dtype=np.uint16)
    alen = np.zeros(B, np.int32)
    path = np.full((B, 64), -1, np.int32)
    for b in range(B):
        chain = [int(rng.integers(0, counts[b]))]
        while parents[b][chain[-1]] >= 0:
            chain.append(int(parents[b][chain[-1]]))
        alen[b] = len(chain)
        path[b, :len(chain)] = chain[::-1]
    return offs, lens, table, k, v, alen, path


@pytest.mark.parametrize("page", [16, 32, 128])
def test_kv_commit_matches_oracle_bit_for_bit(page):
    rng = np.random.default_rng(50 + page)
    for trial in range(6):
        B, hkv = int(rng.integers(1, 6)), int(rng.choice([1, 2, 8]))
        offs, lens, table, k, v, alen, path = _commit_case(rng, B, hkv, page)
        d = make_dims(batch=B, total_nodes=int(offs[-1]), max_nodes=int(np.diff(offs).max()), num_kv_heads=hkv, page_size=page,
                      max_pages_per_seq=table.shape[1], num_pages=k.shape[0])
        ctx = OwlContext(make_dims(batch=B, total_nodes=int(offs[-1]), max_nodes=64))
        kd, vd, ld = dev_bf16(k), dev_bf16(v), dev_i32(lens)
        ctx.owl_kv_commit(d, kd, vd, dev_i32(table), ld, dev_i32(offs), dev_i32(alen), dev_i32(path))
        assert ctx.owl_get_status() == 0
        lens_ref = lens.copy()
        oracle.kv_commit(k, v, table, lens_ref, offs, alen, path)
        np.testing.assert_array_equal(ld.cpu().numpy(), lens_ref)
        assert np.array_equal(bits_of(kd), k) and np.array_equal(bits_of(vd), v)     # the whole cache, dead slots included
        ctx.close()


def test_kv_commit_hand_worked_and_errors(golden_dir):
    g = json.load(open(os.path.join(golden_dir, "kv_commit_cases.json")))
    rng = np.random.default_rng(60)
    ctx = OwlContext(make_dims(batch=4, total_nodes=64, max_nodes=16))
    for case in g["cases"]:
        # the fixture is worked for 4-token pages; what it states - which logical position ends up where - holds for
        # any page size, and the library's smallest page has 16 tokens
        bt = np.asarray(case["block_table"], np.int32)
        B = bt.shape[0]
        k = rng.integers(0, 2 ** 16, size=(int(bt.max()) + 1, 2, 16, 128), dtype=np.uint16)
        v = rng.integers(0, 2 ** 16, size=k.shape, dtype=np.uint16)
        lens = np.asarray(case["ctx_lens"], np.int32)
        offs = np.asarray(case["node_offsets"], np.int32)
        alen, path = np.asarray(case["accept_len"], np.int32), np.asarray(case["accept_path"], np.int32)
        d = make_dims(batch=B, total_nodes=int(offs[-1]), max_nodes=int(np.diff(offs).max()), num_kv_heads=2, page_size=16,
                      max_pages_per_seq=bt.shape[1], num_pages=k.shape[0], path_stride=path.shape[1])
        kd, vd, ld = dev_bf16(k), dev_bf16(v), dev_i32(lens)
        ctx.owl_kv_commit(d, kd, vd, dev_i32(bt), ld, dev_i32(offs), dev_i32(alen), dev_i32(path))
        assert ctx.owl_get_status() == 0
        assert ld.cpu().tolist() == case["new_ctx_lens"]
        for a in case["after"]:
            b, pos, src = a["b"], a["pos"], a["from"]
            assert np.array_equal(bits_of(kd)[bt[b, pos // 16], :, pos % 16], k[bt[b, src // 16], :, src % 16])
            assert np.array_equal(bits_of(vd)[bt[b, pos // 16], :, pos % 16], v[bt[b, src // 16], :, src % 16])
    # a path out of node order in sequence 0 and a page id out of range in sequence 1: both reported (the first
    # error wins the status word), both sequences untouched, sequence 2 committed
    offs = np.array([0, 6, 12, 18], np.int32)
    lens = np.array([10, 12, 10], np.int32)          # sequence 1's drafted positions 12..17 reach its second page
    bt = np.array([[0, 1], [2, 99], [3, 4]], np.int32)
    k = rng.integers(0, 2 ** 16, size=(5, 2, 16, 128), dtype=np.uint16)
    v = rng.integers(0, 2 ** 16, size=k.shape, dtype=np.uint16)
    alen = np.array([3, 2, 3], np.int32)
    path = np.array([[0, 4, 2] + [-1] * 13, [0, 1] + [-1] * 14, [0, 3, 5] + [-1] * 13], np.int32)
    d = make_dims(batch=3, total_nodes=18, max_nodes=6, num_kv_heads=2, page_size=16, max_pages_per_seq=2, num_pages=5, path_stride=16)
    kd, vd, ld = dev_bf16(k), dev_bf16(v), dev_i32(lens)
    ctx.owl_kv_commit(d, kd, vd, dev_i32(bt), ld, dev_i32(offs), dev_i32(alen), dev_i32(path))
    assert ctx.owl_get_status() in (-4, -5)
    assert ld.cpu().tolist() == [10, 12, 13]
    k_ref, v_ref, l_ref = k.copy(), v.copy(), np.array([10], np.int32)
    oracle.kv_commit(k_ref, v_ref, bt[2:3], l_ref, np.array([0, 6], np.int32), alen[2:3], path[2:3])
    assert np.array_equal(bits_of(kd), k_ref) and np.array_equal(bits_of(vd), v_ref)
    # host-detected: nothing launched
    n0 = ctx.launch_count()
    bad = make_dims(batch=3, total_nodes=18, max_nodes=6, num_kv_heads=2, page_size=24, max_pages_per_seq=2, num_pages=5)
    assert ctx.owl_kv_commit(bad, kd, vd, dev_i32(bt), ld, dev_i32(offs), dev_i32(alen), dev_i32(path), check=False) == -2
    assert ctx.owl_kv_commit(d, kd, vd, dev_i32(bt), None, dev_i32(offs), dev_i32(alen), dev_i32(path), check=False) == -1
    assert ctx.launch_count() == n0
    ctx.close()


def test_decoding_loop_200_steps_on_the_device():
    """Algorithm 1 on the toy model.  The cache, the lengths, the prepared trees and the acceptance results live on
    the device for all 200 verification steps (routing -> Prepare on the routed batch -> verify attention ->
    acceptance with [SPEC] pick -> commit); the host only plays the drafter, which gets the next token as a drafter outside the GPU would.  The
    same drafts go through the oracle's loop on the CPU.  Every step's acceptance and lengths must agree, the
    committed text must be the toy model's own (lossless), and at the end the two caches must be the same bits.
    Every 20th step the attention outputs of the step are compared as well."""
    Hq, Hkv, B = 8, 2, 3
    toy_gpu, toy_cpu = W.ToyLoop(batch=B, num_kv_heads=Hkv, seed=23), W.ToyLoop(batch=B, num_kv_heads=Hkv, seed=23)
    k, v = toy_cpu.initial_cache()
    lens = toy_cpu.ctx0.copy()
    kd, vd, ld = dev_bf16(k), dev_bf16(v), dev_i32(lens)
    table_d = dev_i32(toy_gpu.block_table)
    ctx = OwlContext(make_dims(batch=B, total_nodes=64 * B, max_nodes=64, num_q_heads=Hq, num_kv_heads=Hkv,
                               max_pages_per_seq=toy_gpu.max_pages, num_pages=toy_gpu.num_pages, vocab=toy_gpu.V))
    noise_d = torch.from_numpy(toy_gpu.noise).to(DEV)
    roots = [int(toy_cpu.text(b, int(lens[b]) + 1)[-1]) for b in range(B)]
    emitted = [[] for _ in range(B)]
    lastlinear_gpu, lastlinear_cpu = np.zeros(B, np.uint8), np.zeros(B, np.uint8)
    qrng = np.random.default_rng(5)
    for step in range(200):
        kinds, offs, par, tok = toy_gpu.draft(roots)
        kinds2, offs2, par2, tok2 = toy_cpu.draft(roots)
        assert kinds == kinds2 and np.array_equal(tok, tok2)
        N = int(offs[-1])
        # ---- the router (Algorithm 1): the toy non-tree drafter "expects" 30 tokens of its chains, 4 otherwise
        score = np.array([30.0 if kd == "chain" else 4.0 for kd in kinds], np.float32)
        route = owl_howl_route(score, 9.0, lastlinear_gpu)
        np.testing.assert_array_equal(route, oracle.howl_route(score, 9.0, lastlinear_cpu))
        assert [r == 0 for r in route] == [kd == "chain" for kd in kinds]
        # ---- device: Prepare on the routed batch (chains as drafted, trees with their [SPEC] leaves)
        pd = make_dims(batch=B, total_nodes=N, max_nodes=int(np.diff(offs).max()))
        o2 = torch.zeros(B + 1, dtype=torch.int32, device=DEV)
        p2, d2, i2, s2 = (torch.zeros(2 * N, dtype=torch.int32, device=DEV) for _ in range(4))
        ctx.owl_prepare_hybrid(pd, dev_i32(offs), dev_i32(par), dev_i32(tok), ld, dev_i32(route), toy_gpu.spec_token, o2, p2, d2, i2, s2)
        counts = np.array([(1 if kinds[b] == "chain" else 2) * (offs[b + 1] - offs[b]) for b in range(B)])
        v_offs = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
        np.testing.assert_array_equal(o2.cpu().numpy(), v_offs)
        v_offs_d = o2
        Mv = int(v_offs[-1])
        v_par, v_tok, v_ids, v_pos = p2[:Mv].contiguous(), d2[:Mv].contiguous(), i2[:Mv].contiguous(), s2[:Mv].contiguous()
        M = int(v_offs[-1])
        seq_of = torch.from_numpy(np.repeat(np.arange(B), counts)).to(DEV)
        local = torch.from_numpy(np.concatenate([np.arange(c) for c in counts])).to(DEV)
        # the "verifier" writes the drafted nodes' K/V rows (a pattern of token and position id) at slots L + i
        slots = ld[seq_of].long() + local
        pg = table_d[seq_of, slots // toy_gpu.P].long()
        hh = torch.arange(Hkv, device=DEV)[None, :, None]
        dd = torch.arange(128, device=DEV)[None, None, :]
        for which, cache in ((0, kd), (1, vd)):
            x = (v_ids.long()[:, None, None] * 131 + v_pos.long()[:, None, None] * 31 + hh * 7 + which * 3 + dd * 17) % 251 - 125
            cache[pg, :, slots % toy_gpu.P, :] = (x.float() / 64.0).to(torch.bfloat16)
        d = make_dims(batch=B, total_nodes=M, max_nodes=int(counts.max()), num_q_heads=Hq, num_kv_heads=Hkv,
                      max_pages_per_seq=toy_gpu.max_pages, num_pages=toy_gpu.num_pages, vocab=toy_gpu.V, sm_scale=0.25)
        q_bits = W.f32_to_bf16_bits(qrng.standard_normal((M, Hq, 128)).astype(np.float32))
        out = torch.zeros((M, Hq, 128), dtype=torch.bfloat16, device=DEV)
        lse = torch.zeros((M, Hq), dtype=torch.float32, device=DEV)
        ctx.owl_verify_attn(d, dev_bf16(q_bits), kd, vd, table_d, ld, v_offs_d, v_par, out, lse)
        lg = noise_d[:M].clone()
        lg[torch.arange(M, device=DEV), (v_ids.long() * 37 + 11) % toy_gpu.V] += 5.0
        alen = torch.zeros(B, dtype=torch.int32, device=DEV); path = torch.zeros((B, 64), dtype=torch.int32, device=DEV)
        bonus = torch.zeros(B, dtype=torch.int32, device=DEV); leaf = torch.zeros(B, dtype=torch.int32, device=DEV)
        ctx.owl_tree_accept_spec(d, lg, v_tok, v_offs_d, v_par, alen, path, bonus, leaf)
        lens_before_d = ld.clone()
        ctx.owl_kv_commit(d, kd, vd, table_d, ld, v_offs_d, alen, path)
        assert ctx.owl_get_status() == 0

        # ---- the oracle's step on the CPU with the same drafts
        ro2, r_par, r_tok, r_ids, r_pos = oracle.prepare_hybrid(offs, par, tok, lens, route, toy_cpu.spec_token)
        np.testing.assert_array_equal(v_par.cpu().numpy(), r_par)
        np.testing.assert_array_equal(v_pos.cpu().numpy(), r_pos)
        for b in range(B):
            sl = slice(int(v_offs[b]), int(v_offs[b + 1]))
            toy_cpu.write_rows(k, v, b, int(lens[b]) + np.arange(counts[b]), r_ids[sl], r_pos[sl])
        if step % 20 == 0:
            ref_out, ref_lse = oracle.verify_attn(q_bits, k, v, toy_cpu.block_table, lens, v_offs, r_par, 0.25)
            assert np.abs(out.float().cpu().numpy() - ref_out).max() <= 1e-2
            assert np.abs(lse.cpu().numpy() - ref_lse).max() <= 1e-3
        r_alen, r_path, r_bonus, _ = oracle.tree_accept(toy_cpu.logits(r_ids), r_tok, v_offs, r_par, 64)
        r_leaf = oracle.spec_leaf(v_offs, r_par, r_tok, r_alen, r_path)
        oracle.kv_commit(k, v, toy_cpu.block_table, lens, v_offs, r_alen, r_path)
        np.testing.assert_array_equal(alen.cpu().numpy(), r_alen)
        np.testing.assert_array_equal(path.cpu().numpy(), r_path)
        np.testing.assert_array_equal(bonus.cpu().numpy(), r_bonus)
        np.testing.assert_array_equal(leaf.cpu().numpy(), r_leaf)
        np.testing.assert_array_equal(ld.cpu().numpy(), lens)
        np.testing.assert_array_equal((ld - lens_before_d).cpu().numpy(), r_alen)
        for b in range(B):
            emitted[b].extend(int(r_ids[v_offs[b] + j]) for j in r_path[b, :r_alen[b]])
        roots = [int(x) for x in bonus.cpu().numpy()]
    assert np.array_equal(bits_of(kd), k) and np.array_equal(bits_of(vd), v)
    for b in range(B):
        L = int(lens[b])
        text = toy_cpu.text(b, L + 1)
        assert emitted[b] == text[int(toy_cpu.ctx0[b]):L].tolist() and roots[b] == text[L]      # lossless
        pos = np.arange(L)
        assert np.array_equal(toy_cpu.read_rows(bits_of(kd), b, pos), toy_cpu.kv_rows(text[:L], pos, Hkv, 0))
    ctx.close()

"""Parity of the CUDA path (through the C ABI) against the CPU oracle, element by element, on
seeded inputs small enough for the oracle yet spanning several key tiles, ragged tails, several
CTAs per unit and several units per CTA."""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_07535_b200 import OwlContext, make_dims, workloads as W
from paper_2510_07535_b200.runner import DeviceWorkload, dims_of

pytestmark = pytest.mark.gpu

OUT_TOL = 1e-2   # max |err| of the bf16 outputs against the fp64 oracle
LSE_TOL = 1e-3   # max |err| of the fp32 LSE


def check_attention(wl, ctx=None):
    dw = DeviceWorkload.upload(wl)
    own = ctx is None
    ctx = ctx or OwlContext(dims_of(wl))
    dw.attn(ctx)
    assert ctx.owl_get_status() == 0
    ref_out, ref_lse = oracle.verify_attn(wl.q, wl.k_cache, wl.v_cache, wl.block_table, wl.ctx_lens,
                                          wl.node_offsets, wl.tree_parent, wl.sm_scale)
    out, lse = dw.out_f32().astype(np.float64), dw.lse.cpu().numpy().astype(np.float64)
    eo, el = np.abs(out - ref_out).max(), np.abs(lse - ref_lse).max()
    # second run must be bit-identical (no races, no dependence on workspace contents)
    out1 = dw.out.clone(); lse1 = dw.lse.clone()
    dw.out.zero_(); dw.lse.zero_()
    dw.attn(ctx)
    assert torch.equal(out1, dw.out) and torch.equal(lse1, dw.lse)
    if own:
        ctx.close()
    assert eo <= OUT_TOL, f"out err {eo}"
    assert el <= LSE_TOL, f"lse err {el}"
    return eo, el


def check_accept(wl, ctx=None):
    dw = DeviceWorkload.upload(wl)
    own = ctx is None
    ctx = ctx or OwlContext(dims_of(wl))
    for _ in range(2):   # twice: the arg-max scratch must be reset by the call itself
        dw.accept(ctx)
        assert ctx.owl_get_status() == 0
        alen, path, bonus, am = oracle.tree_accept(wl.logits, wl.draft_tokens, wl.node_offsets, wl.tree_parent, 64)
        np.testing.assert_array_equal(dw.node_argmax.cpu().numpy(), am)
        np.testing.assert_array_equal(dw.accept_len.cpu().numpy(), alen)
        np.testing.assert_array_equal(dw.accept_path.cpu().numpy(), path)
        np.testing.assert_array_equal(dw.bonus_token.cpu().numpy(), bonus)
        dw.accept_len.zero_(); dw.accept_path.zero_(); dw.bonus_token.zero_(); dw.node_argmax.zero_()
    if own:
        ctx.close()


@pytest.mark.parametrize("idx", [0, 1, 2, 3, 4])
@pytest.mark.parametrize("prescaled", [True, False])
def test_scaled_down_configs_attention(idx, prescaled):
    """The five benchmark configurations with contexts shrunk 32x-64x (ragged), every output element."""
    div = {0: 4, 1: 32, 2: 128, 3: 64, 4: 64}[idx]
    spec = W.config_spec(idx, ctx_div=div, vocab=1024, q_prescaled=prescaled)
    spec.with_logits = False
    check_attention(W.generate(spec))


@pytest.mark.parametrize("idx", [0, 1, 2, 3, 4])
def test_configs_acceptance_full_vocab(idx):
    """Acceptance at the full vocabulary (128256) of every configuration, bit-exact."""
    spec = W.config_spec(idx, ctx_div=4096)
    check_accept(W.generate(spec))


@pytest.mark.parametrize("hq,hkv,trees,ctx", [
    (8, 8, [("chain", 1)], [1]),                          # G = 1, one node, one context token
    (8, 2, [("chain", 1)], [0]),                          # empty context: the root sees only itself
    (4, 1, [("tree", 64, 8)], [0]),                       # empty context, full 64-node tree (M = 256)
    (32, 8, [("tree", 64, 8), ("chain", 3)], [777, 15]),  # two row blocks + a tiny sequence
    (16, 2, [("tree", 17, 4)] * 3, [63, 64, 65]),         # lengths around a tile edge
    (64, 8, [("tree", 32, 6)], [5000]),                   # 70B head geometry
    (12, 4, [("tree", 11, 4), ("chain", 7)], [300, 1000]),  # G = 3: rows of a node straddle nothing regular
])
def test_edge_shapes_attention(hq, hkv, trees, ctx):
    wl = W.generate(W.Spec("edge", hq, hkv, ctx, trees, shuffle_pages=True, seed=hq * 1000 + ctx[0], with_logits=False))
    check_attention(wl)


def test_draft_keys_straddle_tiles_and_pages():
    # L = 1020: draft positions 1020..1051 cross a 64-key tile edge and a page edge
    wl = W.generate(W.Spec("straddle", 8, 2, [1020, 1080], [("tree", 32, 6), ("tree", 40, 6)], shuffle_pages=True,
                           seed=77, with_logits=False))
    check_attention(wl)


def test_many_short_sequences_one_cta_many_units():
    rng = np.random.default_rng(5)
    ctx = [int(x) for x in rng.integers(1, 200, size=96)]
    trees = [("chain", int(rng.integers(1, 9))) for _ in range(96)]
    wl = W.generate(W.Spec("many", 8, 2, ctx, trees, shuffle_pages=True, seed=78, with_logits=False))
    check_attention(wl)


def test_uniform_node_offsets_null():
    wl = W.generate(W.Spec("uniform", 8, 2, [100, 333, 90], [("tree", 8, 3)] * 3, seed=79, with_logits=True, vocab=1000))
    dw = DeviceWorkload.upload(wl)
    ctx = OwlContext(dims_of(wl))
    dw.node_offsets = None
    dw.step(ctx)
    assert ctx.owl_get_status() == 0
    ref_out, ref_lse = oracle.verify_attn(wl.q, wl.k_cache, wl.v_cache, wl.block_table, wl.ctx_lens,
                                          wl.node_offsets, wl.tree_parent, wl.sm_scale)
    assert np.abs(dw.out_f32() - ref_out).max() <= OUT_TOL
    alen, path, bonus, am = oracle.tree_accept(wl.logits, wl.draft_tokens, wl.node_offsets, wl.tree_parent, 64)
    np.testing.assert_array_equal(dw.accept_len.cpu().numpy(), alen)
    np.testing.assert_array_equal(dw.bonus_token.cpu().numpy(), bonus)
    ctx.close()


@pytest.mark.parametrize("page,hq,hkv,trees,ctx", [
    (16, 8, 2, [("tree", 5, 2)], [22]),                        # 27 keys: 5 dead slots in the second page
    (16, 4, 1, [("tree", 64, 8)], [1000]),                     # 256-row unit (both warpgroups read the tile)
    (64, 16, 4, [("chain", 3), ("tree", 9, 3)], [130, 255]),   # larger pages: up to 63 dead slots
    (128, 8, 2, [("chain", 1)], [128]),                        # one live key in the last 128-token page
])
def test_unused_tail_slots_may_hold_anything(page, hq, hkv, trees, ctx):
    """Slots of a sequence's last page past L + n are never visible: NaN, Inf and huge values there (what
    uninitialised cache memory may hold) must not reach any output.  Same fill as the oracle's own pin."""
    wl = W.generate(W.Spec("tail", hq, hkv, ctx, trees, page_size=page, shuffle_pages=True, seed=80 + page, with_logits=False))
    fills = [0x7FC0, 0x7F80, 0xFF80, 0x7F00]     # NaN, +Inf, -Inf, 1.7e38
    for b in range(wl.spec.batch):
        keys = int(wl.ctx_lens[b]) + int(wl.node_offsets[b + 1] - wl.node_offsets[b])
        last, used = (keys - 1) // page, (keys - 1) % page + 1
        pg = int(wl.block_table[b, last])
        for j in range(used, page):
            wl.k_cache[pg, :, j, :] = fills[j % 4]
            wl.v_cache[pg, :, j, :] = fills[(j + 1) % 4]
    check_attention(wl)


def test_large_scores_stress_relative_tolerance():
    """Outputs of order 10 and scores of order 30: |err| <= 1e-2 + 2^-8 |ref| (bf16 half-ulp dominates)."""
    wl = W.generate(W.Spec("stress", 8, 2, [500], [("tree", 16, 4)], seed=81, with_logits=False, q_prescaled=True))
    v = W.bf16_bits_to_f32(wl.v_cache) * 10
    wl.v_cache[...] = W.f32_to_bf16_bits(v)
    wl.sm_scale = 3.0
    dw = DeviceWorkload.upload(wl)
    ctx = OwlContext(dims_of(wl))
    dw.attn(ctx)
    ref_out, ref_lse = oracle.verify_attn(wl.q, wl.k_cache, wl.v_cache, wl.block_table, wl.ctx_lens,
                                          wl.node_offsets, wl.tree_parent, wl.sm_scale)
    err = np.abs(dw.out_f32() - ref_out)
    assert np.all(err <= 1e-2 + 2.0 ** -8 * np.abs(ref_out)), err.max()
    assert np.abs(dw.lse.cpu().numpy() - ref_lse).max() <= LSE_TOL
    ctx.close()


# ----------------------------------------------------------------------------- acceptance edge cases

def _accept_case(logits, tokens, offsets, parents, stride=64):
    B = len(offsets) - 1
    N = len(parents)
    d = make_dims(batch=B, total_nodes=N, max_nodes=int(np.diff(offsets).max()), vocab=logits.shape[1],
                  path_stride=stride)
    ctx = OwlContext(d)
    dev = "cuda"
    t = lambda a, dt: torch.from_numpy(np.ascontiguousarray(a, dtype=dt)).to(dev)
    alen = torch.zeros(B, dtype=torch.int32, device=dev); path = torch.zeros((B, stride), dtype=torch.int32, device=dev)
    bonus = torch.zeros(B, dtype=torch.int32, device=dev); am = torch.zeros(N, dtype=torch.int32, device=dev)
    ctx.owl_tree_accept(d, t(logits, np.float32), t(tokens, np.int32), t(offsets, np.int32), t(parents, np.int32),
                        alen, path, bonus, am)
    st = ctx.owl_get_status()
    ctx.close()
    return st, alen.cpu().numpy(), path.cpu().numpy(), bonus.cpu().numpy(), am.cpu().numpy()


@pytest.mark.parametrize("V", [1, 2, 3, 5, 8191, 8192, 8193, 8195, 20000, 128256, 128257])
def test_argmax_ragged_vocab_and_special_values(V):
    rng = np.random.default_rng(V)
    N = 9
    lg = rng.standard_normal((N, V)).astype(np.float32)
    if V > 4:
        lg[1, 1] = lg[1, V - 1] = 9.0          # tie -> lower index
        lg[2, :] = -np.inf                      # all -inf -> 0
        lg[3, :] = 0.0; lg[3, 2] = -0.0         # signed zeros tie
        lg[4, 0] = np.nan; lg[4, V // 2] = 30.0  # NaN never wins
        lg[5, :] = np.nan                       # all NaN -> 0
        lg[6, V - 1] = 99.0                     # last element of the row
        lg[7, :] = 1e-41                        # denormals compare exactly
        lg[7, V // 3] = 2e-41
    parents = W.chain_parents(N)
    tokens = rng.integers(0, V, size=N).astype(np.int32)
    st, alen, path, bonus, am = _accept_case(lg, tokens, np.array([0, N]), parents)
    assert st == 0
    r_alen, r_path, r_bonus, r_am = oracle.tree_accept(lg, tokens, np.array([0, N], np.int32), parents, 64)
    np.testing.assert_array_equal(am, r_am)
    np.testing.assert_array_equal(alen, r_alen)
    np.testing.assert_array_equal(path, r_path)
    np.testing.assert_array_equal(bonus, r_bonus)


def test_unaligned_logits_rows():
    """Odd vocabulary: rows start at addresses that are not 16-byte aligned."""
    rng = np.random.default_rng(9)
    V, N = 30001, 12
    lg = rng.standard_normal((N, V)).astype(np.float32)
    lg[np.arange(N), rng.integers(0, V, N)] += 8
    parents = W.random_tree_parents(rng, N, 4)
    tokens = oracle.row_argmax(lg)[np.maximum(parents, 0)].astype(np.int32)   # every edge matches
    tokens[5] = -1                                                            # a [SPEC]-style leaf
    st, alen, path, bonus, am = _accept_case(lg, tokens, np.array([0, N]), parents)
    r = oracle.tree_accept(lg, tokens, np.array([0, N], np.int32), parents, 64)
    assert st == 0
    np.testing.assert_array_equal(am, r[3]); np.testing.assert_array_equal(alen, r[0])
    np.testing.assert_array_equal(path, r[1]); np.testing.assert_array_equal(bonus, r[2])


# ----------------------------------------------------------------------------- other page sizes, fused step

@pytest.mark.parametrize("page", [32, 64, 128])
def test_other_page_sizes(page):
    """One TMA box per (page, head): 8, 16 and 32 KB boxes instead of 4 KB; tails inside a page and a tile."""
    wl = W.generate(W.Spec(f"page{page}", 16, 4, [777, 130, 1], [("tree", 33, 6), ("chain", 8), ("tree", 64, 8)],
                           shuffle_pages=True, page_size=page, seed=300 + page, with_logits=False))
    check_attention(wl)


@pytest.mark.parametrize("vocab", [
    20000,     # rows 16-byte aligned, three chunks per row: the scan rides in the attention kernel's spare warps
    1003,      # rows not 16-byte aligned: scalar head and tail of every chunk
    8193,      # a second chunk of one element
    250000,    # 40 nodes x 31 chunks > 1024 items: the scan follows as a kernel of its own
])
def test_verify_step_equals_the_two_calls(vocab):
    """owl_verify_step (acceptance inside the attention kernels, or after them) gives bit for bit what the two calls give."""
    wl = W.generate(W.Spec("step", 32, 8, [1500, 40], [("tree", 32, 6), ("chain", 8)], shuffle_pages=True, seed=411, vocab=vocab))
    dw = DeviceWorkload.upload(wl)
    ctx = OwlContext(dims_of(wl))
    dw.attn(ctx)
    dw.accept(ctx)
    assert ctx.owl_get_status() == 0
    want = [t.clone() for t in (dw.out, dw.lse, dw.accept_len, dw.accept_path, dw.bonus_token, dw.node_argmax)]
    for _ in range(3):
        for t in (dw.out, dw.lse, dw.accept_len, dw.accept_path, dw.bonus_token, dw.node_argmax):
            t.zero_()
        dw.step(ctx)
        assert ctx.owl_get_status() == 0
        for got, ref in zip((dw.out, dw.lse, dw.accept_len, dw.accept_path, dw.bonus_token, dw.node_argmax), want):
            assert torch.equal(got, ref)
    ctx.close()


# ----------------------------------------------------------------------------- partition and schedule corners

@pytest.mark.parametrize("ctx_len,trees", [
    (3000, [("tree", 32, 6)] * 4),     # uniform batch, 8 units over 148 CTAs: unit-aligned cut, pieces of 1-2 tiles
    (300, [("tree", 32, 6)] * 4),      # fewer tiles per unit than CTAs per unit: most CTAs get nothing
    (5000, [("tree", 64, 8)] * 2),     # uniform, M = 256 (both streams read every tile), aligned cut
    (129, [("chain", 2)] * 3),         # two tiles per unit, second one holds a single key
])
def test_uniform_batches_take_the_aligned_cut(ctx_len, trees):
    wl = W.generate(W.Spec("aligned", 8, 2, [ctx_len] * len(trees), trees, shuffle_pages=True, seed=500 + ctx_len,
                           with_logits=False))
    check_attention(wl)


def test_large_batch_mixed_row_counts():
    """More than 32 sequences (block-wide schedule) with M = 256, M = 128 and tiny units next to one another."""
    rng = np.random.default_rng(6)
    kinds = [("tree", 64, 8), ("tree", 32, 6), ("chain", 3), ("tree", 17, 4)]
    trees = [kinds[int(rng.integers(0, 4))] for _ in range(40)]
    ctx = [int(x) for x in rng.integers(0, 700, size=40)]
    wl = W.generate(W.Spec("mixed40", 16, 4, ctx, trees, shuffle_pages=True, seed=601, with_logits=False))
    check_attention(wl)

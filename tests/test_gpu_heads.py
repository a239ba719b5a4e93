"""The producers either side of the verify step on the GPU, through the C ABI, against the CPU oracle: acceptance
straight from hidden states (LM-head product with the arg-max in its epilogue) and the drafter's LSTM cell (Eq. 1-8)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_07535_b200 import OwlContext, make_dims, workloads as W
from paper_2510_07535_b200.binding import owl_lstm_alpha

pytestmark = pytest.mark.gpu

DEV = "cuda"
dev_i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(DEV)
dev_bf16 = lambda bits: torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(DEV).view(torch.bfloat16)


def _normal_bits(seed, shape, scale=1.0):
    ss = np.random.SeedSequence(seed)
    return W.normal_bf16(ss, int(np.prod(shape)), scale=scale).reshape(shape)


def _oracle_rows(hidden, weight, chunk=16384):
    """Per row: the oracle's arg-max, and the slack tau_row within which fp32 accumulation may rank two logits either
    way, from the oracle's fp64 logits computed vocabulary chunk by chunk (bounded memory)."""
    N, K = hidden.shape
    V = weight.shape[0]
    logits = np.empty((N, V))
    absmax = np.zeros(N)
    ha = np.abs(oracle.decode16(hidden, "bf16").reshape(N, K))
    for v0 in range(0, V, chunk):
        w = weight[v0:v0 + chunk]
        logits[:, v0:v0 + len(w)] = oracle.lm_head_logits(hidden, w)
        absmax = np.maximum(absmax, (ha @ np.abs(oracle.decode16(w, "bf16").reshape(len(w), K)).T).max(axis=1))
    tau = 2.0 * K * 2.0 ** -24 * absmax
    return logits, tau


def _lm_head_case(ctx, seed, trees, K, V, plant=0.7):
    rng = np.random.default_rng(seed)
    parents = [W.chain_parents(t[1]) if t[0] == "chain" else W.random_tree_parents(rng, t[1], t[2]) for t in trees]
    counts = np.array([len(p) for p in parents])
    offs = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
    par = np.concatenate(parents).astype(np.int32)
    N, B = len(par), len(trees)
    hidden = _normal_bits(seed, (N, K))
    weight = _normal_bits(seed + 1, (V, K), scale=1.0 / np.sqrt(K))
    logits, tau = _oracle_rows(hidden, weight)
    am_ref = oracle.row_argmax(logits.astype(np.float32))          # (fp32 rounding of fp64 logits keeps the order up to ties)
    am_ref = np.argmax(logits, axis=1).astype(np.int32)            # first maximum of the fp64 logits
    # drafted tokens: with probability `plant` the target's own continuation of the parent, else another token
    tok = rng.integers(0, V, size=N).astype(np.int32)
    for b in range(B):
        for i in range(1, counts[b]):
            if rng.random() < plant:
                tok[offs[b] + i] = am_ref[offs[b] + par[offs[b] + i]]
    d = make_dims(batch=B, total_nodes=N, max_nodes=int(counts.max()), vocab=V)
    alen = torch.full((B,), -3, dtype=torch.int32, device=DEV); path = torch.full((B, 64), -3, dtype=torch.int32, device=DEV)
    bonus = torch.full((B,), -3, dtype=torch.int32, device=DEV); am = torch.full((N,), -3, dtype=torch.int32, device=DEV)
    hd, wd = dev_bf16(hidden), dev_bf16(weight)
    for _ in range(2):                                             # twice: the keys are cleared by the call itself
        ctx.owl_lm_head_accept(d, hd, wd, dev_i32(tok), dev_i32(offs), dev_i32(par), alen, path, bonus, am)
        assert ctx.owl_get_status() == 0
        am_gpu = am.cpu().numpy()
        rows = np.arange(N)
        # tolerance-aware arg-max: the chosen logit is within tau_row of the row maximum; lowest index on exact ties
        assert np.all(logits[rows, am_gpu] >= logits.max(axis=1) - tau), np.abs(logits[rows, am_gpu] - logits.max(axis=1)).max()
        gap = np.sort(logits, axis=1)[:, -1] - np.sort(logits, axis=1)[:, -2]
        clear = gap > tau
        assert clear.mean() > 0.8          # the test keeps its power: most rows have an unambiguous arg-max
        np.testing.assert_array_equal(am_gpu[clear], am_ref[clear])
        # the walk is integer work: bit for bit what the oracle's walk gives on the same arg-max
        r_alen, r_path, r_bonus = oracle.accept_from_argmax(offs, par, tok, am_gpu, 64)
        np.testing.assert_array_equal(alen.cpu().numpy(), r_alen)
        np.testing.assert_array_equal(path.cpu().numpy(), r_path)
        np.testing.assert_array_equal(bonus.cpu().numpy(), r_bonus)
        if clear.all():
            o_alen, o_path, o_bonus = oracle.accept_from_argmax(offs, par, tok, am_ref, 64)
            np.testing.assert_array_equal(alen.cpu().numpy(), o_alen)
            np.testing.assert_array_equal(bonus.cpu().numpy(), o_bonus)
        alen.fill_(-3); am.fill_(-3)
    return r_alen


@pytest.mark.parametrize("trees,K,V", [
    ([("chain", 8)], 128, 1000),                                    # one row block, ragged last vocabulary tile
    ([("tree", 20, 4), ("chain", 3)], 64, 129),                     # a single k-block; a tile of one column
    ([("tree", 64, 8)] * 3 + [("chain", 8)], 256, 5000),            # 200 rows: two row blocks, double-buffered accumulators
    ([("tree", 64, 8)] * 5, 512, 3000),                             # 320 rows: three row blocks, one accumulator buffer
    ([("tree", 32, 6)], 4096, 20000),                               # the real hidden width: 64 k-blocks per tile
    ([("tree", 64, 8)] * 3, 64, 40000),                             # two row blocks, two rounds of tiles (144 + 128 columns)
    ([("tree", 64, 8)] * 5, 64, 20000),                             # three row blocks, two rounds (80 + 64 columns)
    ([("chain", 5)], 64, 16),                                       # the whole vocabulary is one 16-column tile on one CTA
    ([("tree", 64, 8)] * 2 + [("chain", 2)], 128, 16),              # 130 rows on a CTA pair: one stage per tile, one 16-column tile
    ([("tree", 64, 8)] * 4, 128, 1000),                             # 256 rows on CTA pairs: 63 pairs with a 16-column tile each
    ([("tree", 40, 6)] * 4, 384, 40000),                            # 160 rows on 74 pairs: two rounds (144 + 128 columns), three stages per tile
    ([("tree", 64, 8)] * 6, 128, 40000),                            # 384 rows: three row blocks, K a multiple of 128
    ([("tree", 64, 8)] * 4 + [("chain", 1)], 256, 2000),            # 257 rows: one row in the third row block
])
def test_lm_head_accept_small(trees, K, V):
    ctx = OwlContext(make_dims(batch=8, total_nodes=384, max_nodes=64, vocab=V))
    alen = _lm_head_case(ctx, 1000 + K + V, trees, K, V)
    assert alen.max() > 1
    ctx.close()


def test_lm_head_accept_calls_of_different_sizes_on_one_context():
    """The row keys live in two sets that alternate between calls, each cleared as a whole by the call before: a
    200-row call, an 8-row call, a 200-row call and a 23-row call through one context (two launches each inside
    the helper, so every set is reused after a larger and after a smaller call) all match the oracle."""
    ctx = OwlContext(make_dims(batch=8, total_nodes=384, max_nodes=64, vocab=5000))
    big = [("tree", 64, 8)] * 3 + [("chain", 8)]
    for k, trees in enumerate([big, [("chain", 8)], big, [("tree", 20, 4), ("chain", 3)]]):
        _lm_head_case(ctx, 4000 + k, trees, 128, 5000)
    ctx.close()


def test_lm_head_accept_full_vocabulary():
    """The 8B shape's head: hidden 4096, vocabulary 128256 (1002 column tiles over 148 CTAs), a 32-node tree."""
    ctx = OwlContext(make_dims(batch=1, total_nodes=32, max_nodes=32, vocab=W.VOCAB))
    _lm_head_case(ctx, 77, [("tree", 32, 6)], 4096, W.VOCAB)
    ctx.close()


def test_lm_head_accept_full_vocabulary_on_cta_pairs():
    """Four 64-node trees (256 rows, two row blocks): the product runs on CTA pairs, seven rounds of 256- and 240-column
    tiles over 74 pairs, both accumulator buffers in turn."""
    ctx = OwlContext(make_dims(batch=4, total_nodes=256, max_nodes=64, vocab=W.VOCAB))
    _lm_head_case(ctx, 78, [("tree", 64, 8)] * 4, 4096, W.VOCAB)
    ctx.close()


def test_lm_head_accept_errors():
    ctx = OwlContext(make_dims(batch=8, total_nodes=400, max_nodes=64, vocab=1000))
    one = torch.zeros(400, dtype=torch.int32, device=DEV)
    hid = torch.zeros((400, 96), dtype=torch.bfloat16, device=DEV)
    wt = torch.zeros((1000, 96), dtype=torch.bfloat16, device=DEV)
    n0 = ctx.launch_count()
    d = make_dims(batch=2, total_nodes=16, max_nodes=8, vocab=1000)
    assert ctx.owl_lm_head_accept(d, hid[:16], wt, one, None, one, one, one, one, check=False) == -2      # 96 is no multiple of 64
    d = make_dims(batch=8, total_nodes=400, max_nodes=64, vocab=1000)
    assert ctx.owl_lm_head_accept(d, hid[:, :64].contiguous(), wt[:, :64].contiguous(), one, None, one, one, one, one, check=False) in (-2, -7)
    d = make_dims(batch=2, total_nodes=16, max_nodes=8, vocab=1000)
    assert ctx.owl_lm_head_accept(d, None, wt, one, None, one, one, one, one, check=False) == -1
    assert ctx.launch_count() == n0
    ctx.close()


# ----------------------------------------------------------------------------- drafter cell

def _cell_case(ctx, seed, M, d_in, d, affine, steps=1, z_mean=0.0):
    rng = np.random.default_rng(seed)
    hb = _normal_bits(seed, (M, d_in))
    eb = _normal_bits(seed + 1, (M, d))
    wb = _normal_bits(seed + 2, (4 * d, d_in), scale=1.0 / np.sqrt(d_in))
    alpha = 0.8 if d < 1000 else owl_lstm_alpha(8, d) * 100          # large enough for the embedding to matter
    ln_c = (rng.uniform(0.5, 1.5, d).astype(np.float32), rng.normal(0, 0.2, d).astype(np.float32)) if affine else (None, None)
    ln_z = (rng.uniform(0.5, 1.5, d).astype(np.float32), rng.normal(0, 0.2, d).astype(np.float32)) if affine else (None, None)
    t = lambda a: None if a is None else torch.from_numpy(a).to(DEV)
    z = (z_mean + rng.standard_normal((M, d))).astype(np.float32) if steps == 1 else np.zeros((M, d), np.float32)
    zd = torch.from_numpy(z.copy()).to(DEV)
    hf = torch.zeros((M, d), dtype=torch.float32, device=DEV)
    hb16 = torch.zeros((M, d), dtype=torch.bfloat16, device=DEV)
    ws = torch.empty((M, 4 * d), dtype=torch.float32, device=DEV)
    h_dev = dev_bf16(hb)
    z_ref = z.astype(np.float64)
    h_bits = hb
    for step in range(steps):
        ctx.owl_lstm_cell(h_dev, dev_bf16(eb), dev_bf16(wb), alpha, zd, hf, hb16, ws, (t(ln_c[0]), t(ln_c[1])), (t(ln_z[0]), t(ln_z[1])))
        assert ctx.owl_get_status() == 0
        h_ref, z_ref = oracle.lstm_cell(h_bits, eb, wb.reshape(4, d, d_in), z_ref, alpha, ln_c, ln_z)
        ez = np.abs(zd.cpu().numpy() - z_ref).max()
        eh = np.abs(hf.cpu().numpy() - h_ref).max()
        assert ez <= 2e-3 and eh <= 2e-3, (step, ez, eh)
        hb_ref = hb16.float().cpu().numpy()
        assert np.all(np.abs(hb_ref - h_ref) <= 2e-3 + 2.0 ** -8 * np.abs(h_ref))
        if steps > 1:
            # recurrence (d_in == d): the next step consumes the bf16 h' the device produced; the oracle follows the same bits
            assert d_in == d
            h_bits = hb16.view(torch.int16).cpu().numpy().view(np.uint16)
            h_dev = hb16.clone()
            z_ref = zd.cpu().numpy().astype(np.float64)


@pytest.mark.parametrize("M,d_in,d,affine", [
    (1, 64, 64, False),
    (5, 128, 260, True),            # d no multiple of the column tile: ragged last tile of the product
    (130, 256, 512, True),          # two row blocks
    (300, 64, 128, False),          # three row blocks
    (2, 64, 4, True),               # fewer columns than CTAs in a row's cluster: half of them hold none
    (1, 64, 16384, True),           # the widest cell: four columns per thread, two rounds of product tiles
    (256, 128, 4096, False),        # two full row blocks on CTA pairs, store epilogue, four rounds of 224 / 208 columns
    (129, 384, 36, True),           # one row in the second row block; 144 columns in all
    (300, 256, 512, True),          # three row blocks, store epilogue, K a multiple of 128
])
def test_lstm_cell_small(M, d_in, d, affine):
    ctx = OwlContext(make_dims(batch=1, total_nodes=1, max_nodes=1))
    _cell_case(ctx, 500 + M, M, d_in, d, affine)
    ctx.close()


def test_lstm_cell_state_with_a_large_mean():
    """z ~ +-300 + N(0, 1): z' = z g^f + ... is of the order of a hundred with a non-zero mean, so the second layer
    normalisation works far from the origin (the kernel takes its variance about the mean: per-CTA means and sums of
    squared deviations, combined).  Same tolerance as everywhere; the oracle carries the same z in fp64."""
    ctx = OwlContext(make_dims(batch=1, total_nodes=1, max_nodes=1))
    _cell_case(ctx, 950, 3, 128, 4096, True, z_mean=300.0)
    _cell_case(ctx, 951, 130, 128, 260, False, z_mean=-300.0)
    ctx.close()


def test_lstm_cell_paper_width_and_recurrence():
    """d_in = 4096 -> d = 12288 (Section 4.1), ten drafter states; then three recurrent steps at d_in = d = 1024."""
    ctx = OwlContext(make_dims(batch=1, total_nodes=1, max_nodes=1))
    _cell_case(ctx, 900, 10, 4096, 12288, True)
    _cell_case(ctx, 901, 4, 1024, 1024, False, steps=3)
    ctx.close()


def test_lstm_cell_errors_and_alpha():
    ctx = OwlContext(make_dims(batch=1, total_nodes=1, max_nodes=1))
    assert abs(owl_lstm_alpha(8, 12288) - oracle.lstm_alpha(8, 12288)) < 1e-15
    h = torch.zeros((2, 96), dtype=torch.bfloat16, device=DEV); e = torch.zeros((2, 64), dtype=torch.bfloat16, device=DEV)
    w = torch.zeros((256, 96), dtype=torch.bfloat16, device=DEV); f = torch.zeros((2, 256), dtype=torch.float32, device=DEV)
    n0 = ctx.launch_count()
    assert ctx.owl_lstm_cell(h, e, w, 0.5, f[:, :64].contiguous(), f[:, :64].contiguous(), None, f, check=False) == -2   # d_in = 96
    h64 = torch.zeros((2, 64), dtype=torch.bfloat16, device=DEV); w64 = torch.zeros((256, 64), dtype=torch.bfloat16, device=DEV)
    assert ctx.owl_lstm_cell(h64, e, w64, 0.5, f[:, :64].contiguous(), None, None, f, check=False) == -1                 # no output
    assert ctx.launch_count() == n0
    ctx.close()

"""Seeded synthetic inputs for the verify step (tree-masked attention + greedy acceptance).

This module only *draws inputs*: random K/V/Q tensors, random token trees, random
logits with planted matches, page tables.  It contains none of the method's
arithmetic (no attention, no softmax, no argmax, no acceptance walk), so both the
CPU oracle's tests and the CUDA path's tests may feed from it.

The shapes stand in for the paper's workloads (Llama-3.1-8B / Llama-3.3-70B GQA
geometry, 4K-128K contexts, token trees of a few dozen nodes with depth <= 8 as in
the paper's appendix "Inference Details"); the value distributions are the ones the
benchmark configuration states (K,V ~ N(0,1) in bf16, Q ~ N(0,1)/sqrt(head_dim)).

All tensors are numpy arrays; bf16 tensors are carried as ``uint16`` bit patterns.
"""
from __future__ import annotations

import dataclasses
from concurrent.futures import ThreadPoolExecutor
from typing import List, Optional, Sequence, Tuple

import numpy as np

BASE_SEED = 20251007
PAGE_SIZE = 16
HEAD_DIM = 128
VOCAB = 128256
_CHUNK = 1 << 22  # elements per independently seeded chunk (fixed => thread-count independent)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (round-to-nearest-even), returned as uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    return ((u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _gen(ss: np.random.SeedSequence) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(ss))


def normal_bf16(ss: np.random.SeedSequence, count: int, scale: float = 1.0,
                col_scale: Optional[np.ndarray] = None, threads: int = 8) -> np.ndarray:
    """``count`` N(0,1)*scale samples rounded to bf16 bits.

    ``col_scale`` (length ``HEAD_DIM``) multiplies element ``i`` by ``col_scale[i % HEAD_DIM]``
    before rounding (used for outlier channels; callers pass one vector per call).
    Drawn in fixed-size chunks, each from its own spawned stream, so the result does not
    depend on the number of worker threads.
    """
    out = np.empty(count, dtype=np.uint16)
    nchunks = (count + _CHUNK - 1) // _CHUNK
    children = ss.spawn(max(nchunks, 1))

    def work(c: int) -> None:
        lo = c * _CHUNK
        hi = min(count, lo + _CHUNK)
        x = _gen(children[c]).standard_normal(hi - lo, dtype=np.float32)
        if scale != 1.0:
            x *= np.float32(scale)
        if col_scale is not None:
            assert lo % HEAD_DIM == 0
            x = (x.reshape(-1, HEAD_DIM) * col_scale.astype(np.float32)[None, :]).reshape(-1)
        out[lo:hi] = f32_to_bf16_bits(x)

    if nchunks <= 1 or threads <= 1:
        for c in range(nchunks):
            work(c)
    else:
        with ThreadPoolExecutor(threads) as ex:
            list(ex.map(work, range(nchunks)))
    return out


def normal_f32(ss: np.random.SeedSequence, count: int, threads: int = 8) -> np.ndarray:
    out = np.empty(count, dtype=np.float32)
    nchunks = (count + _CHUNK - 1) // _CHUNK
    children = ss.spawn(max(nchunks, 1))

    def work(c: int) -> None:
        lo = c * _CHUNK
        hi = min(count, lo + _CHUNK)
        _gen(children[c]).standard_normal(out=out[lo:hi], dtype=np.float32)

    if nchunks <= 1 or threads <= 1:
        for c in range(nchunks):
            work(c)
    else:
        with ThreadPoolExecutor(threads) as ex:
            list(ex.map(work, range(nchunks)))
    return out


# --------------------------------------------------------------------------- trees

def chain_parents(n: int) -> np.ndarray:
    """Chain-shaped "tree": node i hangs off node i-1 (non-tree verification)."""
    return np.arange(-1, n - 1, dtype=np.int32)


def random_tree_parents(rng: np.random.Generator, n: int, max_depth: int,
                        max_children: int = 4) -> np.ndarray:
    """BFS-ordered random tree with exactly ``n`` nodes.

    Nodes are expanded in index order; a node of depth < ``max_depth`` draws
    c ~ U{1..max_children} children, until ``n`` nodes exist.  If the frontier
    empties first the draw is repeated.  ``parent[i] < i``, node 0 is the only root.
    """
    if n == 1:
        return np.array([-1], dtype=np.int32)
    if n > (max_children ** (max_depth + 1) - 1) // (max_children - 1):
        raise ValueError(f"{n} nodes cannot fit in depth {max_depth} with <= {max_children} children per node")
    while True:
        parent = [-1]
        depth = [0]
        i = 0
        while len(parent) < n and i < len(parent):
            if depth[i] < max_depth:
                c = int(rng.integers(1, max_children + 1))
                for _ in range(c):
                    if len(parent) >= n:
                        break
                    parent.append(i)
                    depth.append(depth[i] + 1)
            i += 1
        if len(parent) == n:
            return np.asarray(parent, dtype=np.int32)


def tree_depths(parent: Sequence[int]) -> np.ndarray:
    d = np.zeros(len(parent), dtype=np.int32)
    for i, p in enumerate(parent):
        d[i] = 0 if p < 0 else d[p] + 1
    return d


# --------------------------------------------------------------------------- spec

@dataclasses.dataclass
class Spec:
    """Shape recipe of one workload.  ``trees[b]`` is ("chain", n) or ("tree", n, max_depth)."""
    name: str
    num_q_heads: int
    num_kv_heads: int
    ctx_lens: List[int]
    trees: List[Tuple]
    shuffle_pages: bool = False
    k_outliers: bool = False
    plant_prob: float = 0.7
    vocab: int = VOCAB
    head_dim: int = HEAD_DIM
    page_size: int = PAGE_SIZE
    # True: Q ~ N(0,1)/sqrt(D) with sm_scale = 1 (scale folded into Q);
    # False: Q ~ N(0,1) with sm_scale = 1/sqrt(D) (Llama form).
    q_prescaled: bool = True
    seed: int = BASE_SEED
    with_logits: bool = True

    @property
    def batch(self) -> int:
        return len(self.ctx_lens)

    def node_counts(self) -> List[int]:
        return [t[1] for t in self.trees]

    def kv_bytes(self) -> int:
        """K+V bytes of all visible positions (prefix + draft slots), all KV heads."""
        keys = sum(l + n for l, n in zip(self.ctx_lens, self.node_counts()))
        return keys * self.num_kv_heads * self.head_dim * 2 * 2

    def logits_bytes(self) -> int:
        return sum(self.node_counts()) * self.vocab * 4


@dataclasses.dataclass
class Workload:
    spec: Spec
    q: np.ndarray             # uint16 [N, Hq, D] (bf16 bits)
    k_cache: np.ndarray       # uint16 [num_pages, Hkv, page, D]
    v_cache: np.ndarray       # uint16 same
    block_table: np.ndarray   # int32 [B, max_pages_per_seq]
    ctx_lens: np.ndarray      # int32 [B]
    node_offsets: np.ndarray  # int32 [B+1]
    tree_parent: np.ndarray   # int32 [N] (local indices, -1 = root)
    draft_tokens: np.ndarray  # int32 [N]
    logits: Optional[np.ndarray]  # float32 [N, V]
    sm_scale: float

    @property
    def total_nodes(self) -> int:
        return int(self.node_offsets[-1])

    @property
    def max_nodes(self) -> int:
        return int(np.max(np.diff(self.node_offsets)))

    @property
    def num_pages(self) -> int:
        return int(self.k_cache.shape[0])

    @property
    def max_pages_per_seq(self) -> int:
        return int(self.block_table.shape[1])


def generate(spec: Spec, threads: int = 8) -> Workload:
    """Draw every tensor of ``spec`` from its own stream spawned off ``spec.seed``."""
    B, Hq, Hkv, D, P = spec.batch, spec.num_q_heads, spec.num_kv_heads, spec.head_dim, spec.page_size
    assert D == HEAD_DIM
    root = np.random.SeedSequence(spec.seed)
    s_tree, s_q, s_k, s_v, s_tab, s_tok, s_logit, s_plant, s_out = root.spawn(9)

    # trees
    tree_rngs = [_gen(s) for s in s_tree.spawn(B)]
    parents = []
    for b, t in enumerate(spec.trees):
        if t[0] == "chain":
            parents.append(chain_parents(t[1]))
        else:
            parents.append(random_tree_parents(tree_rngs[b], t[1], t[2]))
    counts = np.array([len(p) for p in parents], dtype=np.int64)
    node_offsets = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
    N = int(node_offsets[-1])
    tree_parent = np.concatenate(parents).astype(np.int32)

    # pages
    ctx = np.asarray(spec.ctx_lens, dtype=np.int64)
    pages_per_seq = (ctx + counts + P - 1) // P
    num_pages = int(pages_per_seq.sum())
    max_pages = int(pages_per_seq.max())
    order = np.arange(num_pages, dtype=np.int32)
    if spec.shuffle_pages:
        order = _gen(s_tab).permutation(num_pages).astype(np.int32)
    block_table = np.zeros((B, max_pages), dtype=np.int32)
    o = 0
    for b in range(B):
        block_table[b, :pages_per_seq[b]] = order[o:o + pages_per_seq[b]]
        o += int(pages_per_seq[b])

    # Q / K / V
    q_scale = 1.0 / np.sqrt(D) if spec.q_prescaled else 1.0
    sm_scale = 1.0 if spec.q_prescaled else 1.0 / float(np.sqrt(D))
    q = normal_bf16(s_q, N * Hq * D, scale=q_scale, threads=threads).reshape(N, Hq, D)
    kv_elems = num_pages * Hkv * P * D
    if spec.k_outliers:
        # per KV head, ceil(0.01*D) channel indices fixed over tokens, K scaled x20 there
        n_out = int(np.ceil(0.01 * D))
        g = _gen(s_out)
        col = np.ones((Hkv, D), dtype=np.float32)
        for h in range(Hkv):
            col[h, g.choice(D, size=n_out, replace=False)] = 20.0
        k_cache = np.empty((num_pages, Hkv, P, D), dtype=np.uint16)
        # one draw per head keeps the column pattern constant inside a call
        for h, s in enumerate(s_k.spawn(Hkv)):
            k_cache[:, h] = normal_bf16(s, num_pages * P * D, col_scale=col[h], threads=threads).reshape(num_pages, P, D)
    else:
        k_cache = normal_bf16(s_k, kv_elems, threads=threads).reshape(num_pages, Hkv, P, D)
    v_cache = normal_bf16(s_v, kv_elems, threads=threads).reshape(num_pages, Hkv, P, D)

    # draft tokens: distinct among siblings
    g = _gen(s_tok)
    draft_tokens = np.zeros(N, dtype=np.int32)
    for b in range(B):
        par = parents[b]
        base = int(node_offsets[b])
        draft_tokens[base] = int(g.integers(0, spec.vocab))
        kids = {}
        for i in range(1, len(par)):
            kids.setdefault(int(par[i]), []).append(i)
        for p, ch in kids.items():
            toks = g.choice(spec.vocab, size=len(ch), replace=False)
            for i, t in zip(ch, toks):
                draft_tokens[base + i] = int(t)

    logits = None
    if spec.with_logits:
        logits = normal_f32(s_logit, N * spec.vocab, threads=threads).reshape(N, spec.vocab)
        g = _gen(s_plant)
        for b in range(B):
            par = parents[b]
            base = int(node_offsets[b])
            hit = g.random(len(par)) < spec.plant_prob
            for i in range(1, len(par)):
                if hit[i]:
                    logits[base + int(par[i]), draft_tokens[base + i]] += np.float32(10.0)

    return Workload(spec=spec, q=q, k_cache=k_cache, v_cache=v_cache, block_table=block_table,
                    ctx_lens=ctx.astype(np.int32), node_offsets=node_offsets, tree_parent=tree_parent,
                    draft_tokens=draft_tokens, logits=logits, sm_scale=sm_scale)


# --------------------------------------------------------------------------- the five configurations

def config_spec(idx: int, ctx_div: int = 1, vocab: Optional[int] = None, q_prescaled: bool = True) -> Spec:
    """Benchmark configuration ``idx`` (0..4).

    ``ctx_div`` > 1 shrinks every context length by that factor (ragged tails are
    kept by adding a small odd offset) for element-by-element parity runs the CPU
    oracle can finish in seconds; ``vocab`` overrides the vocabulary likewise.
    """
    V = VOCAB if vocab is None else vocab
    seed = BASE_SEED + idx

    def L(x: int, k: int = 0) -> int:
        return x if ctx_div == 1 else max(17, x // ctx_div + 3 + 5 * k)

    if idx == 0:
        return Spec("cfg0_8b_2k_chain8", 32, 8, [L(2048)], [("chain", 8)], plant_prob=0.7, vocab=V,
                    seed=seed, q_prescaled=q_prescaled)
    if idx == 1:
        return Spec("cfg1_8b_32k_tree32", 32, 8, [L(32768)], [("tree", 32, 6)], plant_prob=0.7, vocab=V,
                    seed=seed, q_prescaled=q_prescaled)
    if idx == 2:
        return Spec("cfg2_8b_4x128k_tree64_paged", 32, 8, [L(131072, b) for b in range(4)],
                    [("tree", 64, 8)] * 4, shuffle_pages=True, plant_prob=0.6, vocab=V, seed=seed,
                    q_prescaled=q_prescaled)
    if idx == 3:
        return Spec("cfg3_70b_8x64k_tree32", 64, 8, [L(65536, b) for b in range(8)],
                    [("tree", 32, 6)] * 8, k_outliers=True, plant_prob=0.7, vocab=V, seed=seed,
                    q_prescaled=q_prescaled)
    if idx == 4:
        g = _gen(np.random.SeedSequence(seed).spawn(10)[9])
        lens = g.integers(4096, 131072 + 1, size=16)
        kinds = [("chain", 8)] * 8 + [("tree", 32, 6)] * 8
        perm = g.permutation(16)
        kinds = [kinds[i] for i in perm]
        ctx = [L(int(x), b) for b, x in enumerate(lens)]
        return Spec("cfg4_8b_16xmixed_hybrid", 32, 8, ctx, kinds, shuffle_pages=True, plant_prob=0.65,
                    vocab=V, seed=seed, q_prescaled=q_prescaled)
    raise ValueError(f"no such configuration: {idx}")


# --------------------------------------------------------------------------- toy decoding loop (inputs only)

class ToyLoop:
    """Inputs of a multi-step speculative-decoding loop on a toy "language model".

    The toy model is a fixed map ``f`` on token ids: the text of sequence b is s_0, s_1 = f(s_0), ... and the
    target's logits row for a node holding token t has its maximum at f(t).  Every step draws, per sequence, a
    chain (verified without [SPEC]) or a tree (verified with one [SPEC] leaf per node), whose drafted tokens are
    right (= f of the parent's token) with probability ``p_right`` and wrong otherwise, at most one right child
    per parent and all siblings distinct.  K/V rows are a fixed pattern of (token, position id, head), so that a
    cache can be checked against the text it should hold.  Nothing here verifies, accepts or commits anything.
    """

    def __init__(self, batch: int, vocab: int = 1000, num_kv_heads: int = 2, page_size: int = PAGE_SIZE,
                 ctx0: Sequence[int] = (), max_tokens: int = 2048, p_right: float = 0.7, spec_token: int = 999,
                 seed: int = 7):
        self.B, self.V, self.Hkv, self.P = batch, vocab, num_kv_heads, page_size
        self.spec_token, self.p_right = spec_token, p_right
        self.rng = _gen(np.random.SeedSequence(seed))
        self.ctx0 = np.asarray(ctx0 if len(ctx0) else self.rng.integers(1, 40, size=batch), dtype=np.int32)
        self.start = self.rng.integers(0, vocab, size=batch)
        self.max_pages = (max_tokens + page_size - 1) // page_size
        self.num_pages = batch * self.max_pages
        self.block_table = self.rng.permutation(self.num_pages).astype(np.int32).reshape(batch, self.max_pages)
        self.noise = self.rng.random((64 * batch, vocab), dtype=np.float32)

    def f(self, t):
        """The toy model's next token (works on ints and integer arrays)."""
        return (t * 37 + 11) % self.V

    def text(self, b: int, length: int) -> np.ndarray:
        out = np.empty(length, dtype=np.int64)
        t = int(self.start[b])
        for j in range(length):
            out[j] = t
            t = int(self.f(t))
        return out

    @staticmethod
    def kv_rows(tokens, positions, num_kv_heads: int, which: int) -> np.ndarray:
        """bf16 bit patterns [len, Hkv, 128] of the K (which = 0) or V (1) rows of tokens at position ids."""
        t = np.asarray(tokens, dtype=np.int64)[:, None, None]
        p = np.asarray(positions, dtype=np.int64)[:, None, None]
        h = np.arange(num_kv_heads, dtype=np.int64)[None, :, None]
        d = np.arange(HEAD_DIM, dtype=np.int64)[None, None, :]
        x = (t * 131 + p * 31 + h * 7 + which * 3 + d * 17) % 251 - 125
        return f32_to_bf16_bits((x / 64.0).astype(np.float32))   # multiples of 1/64 below 2: exact in bf16

    def initial_cache(self):
        """Caches holding the first ctx0[b] tokens of every text; everything else is a recognisable filler."""
        k = np.full((self.num_pages, self.Hkv, self.P, HEAD_DIM), 0x3F80, dtype=np.uint16)
        v = np.full_like(k, 0x3F80)
        for b in range(self.B):
            L = int(self.ctx0[b])
            pos = np.arange(L)
            self.write_rows(k, v, b, pos, self.text(b, L), pos)
        return k, v

    def write_rows(self, k_cache, v_cache, b: int, slots, tokens, positions) -> None:
        """Stores the rows of `tokens` (with position ids `positions`) at logical slots `slots` of sequence b."""
        slots = np.asarray(slots, dtype=np.int64)
        pg = self.block_table[b, slots // self.P]
        k_cache[pg, :, slots % self.P, :] = self.kv_rows(tokens, positions, self.Hkv, 0)
        v_cache[pg, :, slots % self.P, :] = self.kv_rows(tokens, positions, self.Hkv, 1)

    def read_rows(self, cache, b: int, slots) -> np.ndarray:
        slots = np.asarray(slots, dtype=np.int64)
        return cache[self.block_table[b, slots // self.P], :, slots % self.P, :]

    def draft(self, roots: Sequence[int]):
        """One step's drafts: (kinds, node_offsets, tree_parent, draft_tokens); kinds[b] is "chain" or "tree"."""
        kinds, parents, tokens = [], [], []
        for b in range(self.B):
            if self.rng.random() < 0.35:
                kinds.append("chain")
                par = chain_parents(int(self.rng.integers(1, 9)))
            else:
                kinds.append("tree")
                par = random_tree_parents(self.rng, int(self.rng.integers(1, 31)), 8)
            tok = np.zeros(len(par), dtype=np.int64)
            tok[0] = int(roots[b])
            kids = {}
            for i in range(1, len(par)):
                kids.setdefault(int(par[i]), []).append(i)
            for p_, ch in kids.items():               # parents come in increasing order: tok[p_] is final
                right = int(self.f(tok[p_]))
                lucky = int(self.rng.integers(0, len(ch))) if self.rng.random() < self.p_right else -1
                wrong = 0
                for j, i in enumerate(ch):
                    if j == lucky:
                        tok[i] = right
                    else:
                        wrong += 1
                        tok[i] = (right + wrong) % self.V
            parents.append(par)
            tokens.append(tok)
        counts = np.array([len(p_) for p_ in parents])
        offsets = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
        return kinds, offsets, np.concatenate(parents).astype(np.int32), np.concatenate(tokens).astype(np.int32)

    def logits(self, input_ids) -> np.ndarray:
        """fp32 [len, V]: fixed noise in [0, 1) plus 5 at f(token) of every row's token."""
        ids = np.asarray(input_ids, dtype=np.int64)
        lg = self.noise[:len(ids)].copy()
        lg[np.arange(len(ids)), self.f(ids)] += np.float32(5.0)
        return lg

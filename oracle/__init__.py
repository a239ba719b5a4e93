"""ctypes front end of the CPU oracle (``owl_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the
benchmark's CPU-baseline leg.  The CUDA library and its Python binding never
import this package, and this package never imports them.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "owl_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile ``owl_oracle.c`` with gcc (-O2, OpenMP) into ``liboracle.so`` beside it."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        i32p = ctypes.POINTER(ctypes.c_int32)
        u16p = ctypes.POINTER(ctypes.c_uint16)
        f64p = ctypes.POINTER(ctypes.c_double)
        lib.owl_oracle_attn.restype = ctypes.c_int
        lib.owl_oracle_attn.argtypes = [ctypes.c_int] * 7 + [ctypes.c_double, u16p, u16p, u16p, i32p, i32p, i32p, i32p,
                                                              ctypes.c_int64, i32p, i32p, f64p, f64p]
        lib.owl_oracle_attn_f16.restype = ctypes.c_int
        lib.owl_oracle_attn_f16.argtypes = lib.owl_oracle_attn.argtypes
        lib.owl_oracle_decode16.restype = None
        lib.owl_oracle_decode16.argtypes = [u16p, ctypes.c_int64, ctypes.c_int, f64p]
        lib.owl_oracle_howl_route.restype = None
        lib.owl_oracle_howl_route.argtypes = [ctypes.c_int, ctypes.POINTER(ctypes.c_float), ctypes.c_float,
                                              ctypes.POINTER(ctypes.c_uint8), i32p]
        lib.owl_oracle_prepare_hybrid.restype = ctypes.c_int
        lib.owl_oracle_prepare_hybrid.argtypes = [ctypes.c_int, i32p, i32p, i32p, i32p, i32p, ctypes.c_int32] + [i32p] * 5
        lib.owl_oracle_argmax.restype = None
        lib.owl_oracle_argmax.argtypes = [ctypes.POINTER(ctypes.c_float), ctypes.c_int64, ctypes.c_int64, i32p]
        lib.owl_oracle_accept.restype = ctypes.c_int
        lib.owl_oracle_accept.argtypes = [ctypes.c_int, i32p, i32p, i32p, i32p, ctypes.c_int, i32p, i32p, i32p]
        lib.owl_oracle_num_threads.restype = ctypes.c_int
        lib.owl_oracle_prepare_spec.restype = ctypes.c_int
        lib.owl_oracle_prepare_spec.argtypes = [ctypes.c_int, i32p, i32p, i32p, i32p, ctypes.c_int32] + [i32p] * 5
        lib.owl_oracle_spec_leaf.restype = ctypes.c_int
        lib.owl_oracle_spec_leaf.argtypes = [ctypes.c_int, i32p, i32p, i32p, i32p, i32p, ctypes.c_int, i32p]
        lib.owl_oracle_kv_commit.restype = ctypes.c_int
        lib.owl_oracle_kv_commit.argtypes = [ctypes.c_int] * 6 + [u16p, u16p, i32p, i32p, i32p, i32p, i32p, ctypes.c_int]
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().owl_oracle_num_threads())


def _p(a: Optional[np.ndarray], ct):
    if a is None:
        return None
    return a.ctypes.data_as(ctypes.POINTER(ct))


def _c(a, dtype) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def verify_attn(q, k_cache, v_cache, block_table, ctx_lens, node_offsets, tree_parent, sm_scale: float,
                rows: Optional[Tuple[np.ndarray, np.ndarray]] = None, dtype: str = "bf16") -> Tuple[np.ndarray, np.ndarray]:
    """Tree-masked attention in fp64.  ``dtype``: how the 16-bit patterns of q / k_cache / v_cache read, "bf16" or "f16".

    q uint16 [N,Hq,D] (bf16 bits); k_cache/v_cache uint16 [pages,Hkv,page,D]; block_table int32
    [B,max_pages]; ctx_lens int32 [B]; node_offsets int32 [B+1]; tree_parent int32 [N].
    Returns (out, lse): without ``rows`` shapes [N,Hq,D] and [N,Hq]; with
    ``rows=(nodes, heads)`` shapes [R,D] and [R] for the listed (packed node, query head) pairs.
    """
    lib = _load()
    q = _c(q, np.uint16); k_cache = _c(k_cache, np.uint16); v_cache = _c(v_cache, np.uint16)
    block_table = _c(block_table, np.int32); ctx_lens = _c(ctx_lens, np.int32)
    node_offsets = _c(node_offsets, np.int32); tree_parent = _c(tree_parent, np.int32)
    N, Hq, D = q.shape
    num_pages, Hkv, page, D2 = k_cache.shape
    assert D2 == D and v_cache.shape == k_cache.shape
    B = ctx_lens.shape[0]
    assert block_table.shape[0] == B and node_offsets.shape[0] == B + 1 and int(node_offsets[-1]) == N
    if rows is None:
        n_rows = N * Hq
        rn = rh = None
        out = np.empty((N, Hq, D), dtype=np.float64)
        lse = np.empty((N, Hq), dtype=np.float64)
    else:
        rn = _c(rows[0], np.int32); rh = _c(rows[1], np.int32)
        n_rows = rn.shape[0]
        assert rh.shape[0] == n_rows
        out = np.empty((n_rows, D), dtype=np.float64)
        lse = np.empty((n_rows,), dtype=np.float64)
    fn = {"bf16": lib.owl_oracle_attn, "f16": lib.owl_oracle_attn_f16}[dtype]
    rc = fn(B, Hq, Hkv, D, page, block_table.shape[1], num_pages, float(sm_scale),
                             _p(q, ctypes.c_uint16), _p(k_cache, ctypes.c_uint16), _p(v_cache, ctypes.c_uint16),
                             _p(block_table, ctypes.c_int32), _p(ctx_lens, ctypes.c_int32),
                             _p(node_offsets, ctypes.c_int32), _p(tree_parent, ctypes.c_int32),
                             n_rows, _p(rn, ctypes.c_int32), _p(rh, ctypes.c_int32),
                             _p(out, ctypes.c_double), _p(lse, ctypes.c_double))
    if rc != 0:
        raise ValueError(f"owl_oracle_attn failed with code {rc}")
    return out, lse


def row_argmax(logits) -> np.ndarray:
    """Lowest index of the maximum of every row of fp32 ``logits`` [N,V]."""
    lib = _load()
    logits = _c(logits, np.float32)
    N, V = logits.shape
    am = np.empty(N, dtype=np.int32)
    lib.owl_oracle_argmax(_p(logits, ctypes.c_float), N, V, _p(am, ctypes.c_int32))
    return am


def accept_from_argmax(node_offsets, tree_parent, draft_tokens, am, path_stride: int = 64):
    """Greedy tree acceptance given per-node arg-max tokens. Returns (accept_len, accept_path, bonus)."""
    lib = _load()
    node_offsets = _c(node_offsets, np.int32); tree_parent = _c(tree_parent, np.int32)
    draft_tokens = _c(draft_tokens, np.int32); am = _c(am, np.int32)
    B = node_offsets.shape[0] - 1
    alen = np.empty(B, dtype=np.int32)
    path = np.empty((B, path_stride), dtype=np.int32)
    bonus = np.empty(B, dtype=np.int32)
    rc = lib.owl_oracle_accept(B, _p(node_offsets, ctypes.c_int32), _p(tree_parent, ctypes.c_int32),
                               _p(draft_tokens, ctypes.c_int32), _p(am, ctypes.c_int32), path_stride,
                               _p(alen, ctypes.c_int32), _p(path, ctypes.c_int32), _p(bonus, ctypes.c_int32))
    if rc != 0:
        raise ValueError(f"owl_oracle_accept failed with code {rc}")
    return alen, path, bonus


def tree_accept(logits, draft_tokens, node_offsets, tree_parent, path_stride: int = 64):
    """Row arg-max followed by the acceptance walk. Returns (accept_len, accept_path, bonus, argmax)."""
    am = row_argmax(logits)
    alen, path, bonus = accept_from_argmax(node_offsets, tree_parent, draft_tokens, am, path_stride)
    return alen, path, bonus, am


def prepare_spec_tree(node_offsets, tree_parent, draft_tokens, ctx_lens, spec_token: int):
    """Prepare(d): one [SPEC] leaf after every tree path.  Returns (node_offsets, tree_parent, draft_tokens,
    input_ids, position_ids) of the augmented trees (twice the nodes; leaves carry draft token -1)."""
    lib = _load()
    node_offsets = _c(node_offsets, np.int32); tree_parent = _c(tree_parent, np.int32)
    draft_tokens = _c(draft_tokens, np.int32); ctx_lens = _c(ctx_lens, np.int32)
    B = node_offsets.shape[0] - 1
    N = int(node_offsets[-1])
    offs = np.empty(B + 1, np.int32)
    par, drf, ids, pos = (np.empty(2 * N, np.int32) for _ in range(4))
    i32 = ctypes.c_int32
    rc = lib.owl_oracle_prepare_spec(B, _p(node_offsets, i32), _p(tree_parent, i32), _p(draft_tokens, i32), _p(ctx_lens, i32),
                                     int(spec_token), _p(offs, i32), _p(par, i32), _p(drf, i32), _p(ids, i32), _p(pos, i32))
    if rc != 0:
        raise ValueError(f"owl_oracle_prepare_spec failed with code {rc}")
    return offs, par, drf, ids, pos


def spec_leaf(node_offsets, tree_parent, draft_tokens, accept_len, accept_path) -> np.ndarray:
    """Index of the [SPEC] leaf hanging off the last accepted node of every sequence (-1 if none)."""
    lib = _load()
    node_offsets = _c(node_offsets, np.int32); tree_parent = _c(tree_parent, np.int32)
    draft_tokens = _c(draft_tokens, np.int32); accept_len = _c(accept_len, np.int32); accept_path = _c(accept_path, np.int32)
    B = node_offsets.shape[0] - 1
    out = np.empty(B, np.int32)
    i32 = ctypes.c_int32
    rc = lib.owl_oracle_spec_leaf(B, _p(node_offsets, i32), _p(tree_parent, i32), _p(draft_tokens, i32), _p(accept_len, i32),
                                  _p(accept_path, i32), accept_path.shape[1], _p(out, i32))
    if rc != 0:
        raise ValueError(f"owl_oracle_spec_leaf failed with code {rc}")
    return out


def kv_commit(k_cache, v_cache, block_table, ctx_lens, node_offsets, accept_len, accept_path) -> None:
    """Moves the accepted nodes' K/V from L + path[k] to L + k and adds accept_len to ctx_lens, IN PLACE
    (k_cache, v_cache: contiguous uint16 [pages, Hkv, page, D]; ctx_lens: contiguous int32 [B])."""
    lib = _load()
    for a, dt in ((k_cache, np.uint16), (v_cache, np.uint16), (ctx_lens, np.int32)):
        assert a.dtype == dt and a.flags["C_CONTIGUOUS"], "in-place arguments must be contiguous arrays of the exact type"
    block_table = _c(block_table, np.int32); node_offsets = _c(node_offsets, np.int32)
    accept_len = _c(accept_len, np.int32); accept_path = _c(accept_path, np.int32)
    num_pages, Hkv, page, D = k_cache.shape
    B = ctx_lens.shape[0]
    i32, u16 = ctypes.c_int32, ctypes.c_uint16
    rc = lib.owl_oracle_kv_commit(B, Hkv, D, page, block_table.shape[1], num_pages, _p(k_cache, u16), _p(v_cache, u16),
                                  _p(block_table, i32), _p(ctx_lens, i32), _p(node_offsets, i32), _p(accept_len, i32),
                                  _p(accept_path, i32), accept_path.shape[1])
    if rc != 0:
        raise ValueError(f"owl_oracle_kv_commit failed with code {rc}")


def decode16(bits, dtype: str) -> np.ndarray:
    """The oracle's own decoding of 16-bit patterns ("bf16" or "f16") to float64."""
    lib = _load()
    bits = _c(bits, np.uint16).ravel()
    out = np.empty(bits.shape[0], np.float64)
    lib.owl_oracle_decode16(_p(bits, ctypes.c_uint16), bits.shape[0], 1 if dtype == "f16" else 0, _p(out, ctypes.c_double))
    return out


def howl_route(score, c: float, lastwaslinear: np.ndarray) -> np.ndarray:
    """Algorithm 1's routing for one step; ``lastwaslinear`` (uint8 [B]) is updated in place.
    Returns route [B]: 0 = linear (non-tree) verification, 1 = tree from D_nospec, 2 = tree from D_spec."""
    lib = _load()
    score = _c(score, np.float32)
    assert lastwaslinear.dtype == np.uint8 and lastwaslinear.flags["C_CONTIGUOUS"]
    route = np.empty(score.shape[0], np.int32)
    lib.owl_oracle_howl_route(score.shape[0], _p(score, ctypes.c_float), float(c), _p(lastwaslinear, ctypes.c_uint8),
                              _p(route, ctypes.c_int32))
    return route


def prepare_hybrid(node_offsets, tree_parent, draft_tokens, ctx_lens, route, spec_token: int):
    """Prepare(d) on a routed batch (route 0: chain as drafted; else [SPEC] leaves appended).  Returns
    (node_offsets, tree_parent, draft_tokens, input_ids, position_ids) of the batch to verify."""
    lib = _load()
    node_offsets = _c(node_offsets, np.int32); tree_parent = _c(tree_parent, np.int32)
    draft_tokens = _c(draft_tokens, np.int32); ctx_lens = _c(ctx_lens, np.int32); route = _c(route, np.int32)
    B = node_offsets.shape[0] - 1
    N = int(node_offsets[-1])
    offs = np.empty(B + 1, np.int32)
    par, drf, ids, pos = (np.empty(2 * N, np.int32) for _ in range(4))
    i32 = ctypes.c_int32
    rc = lib.owl_oracle_prepare_hybrid(B, _p(node_offsets, i32), _p(tree_parent, i32), _p(draft_tokens, i32), _p(ctx_lens, i32),
                                       _p(route, i32), int(spec_token), _p(offs, i32), _p(par, i32), _p(drf, i32), _p(ids, i32),
                                       _p(pos, i32))
    if rc != 0:
        raise ValueError(f"owl_oracle_prepare_hybrid failed with code {rc}")
    M = int(offs[-1])
    return offs, par[:M], drf[:M], ids[:M], pos[:M]


# ----------------------------------------------------------------------------- the steps either side of the path

def lm_head_logits(hidden_bits, weight_bits) -> np.ndarray:
    """Logits of the verifier's LM head in fp64: hidden (bf16 bits [N, K]) times weight^T (bf16 bits [V, K]).
    A library matrix product of the exactly decoded operands; nothing else."""
    h = decode16(hidden_bits, "bf16").reshape(np.shape(hidden_bits))
    w = decode16(weight_bits, "bf16").reshape(np.shape(weight_bits))
    return h @ w.T


def lstm_alpha(n_depth: int, d: int) -> float:
    """The embedding weight of Eq. 3-4: alpha_0 = 2^(-1/(2n)), alpha = 2 alpha_0 / ((1 - alpha_0^2) d)."""
    a0 = 2.0 ** (-1.0 / (2.0 * n_depth))
    return 2.0 * a0 / ((1.0 - a0 * a0) * d)


def _layer_norm_gelu(x: np.ndarray, gamma, beta, eps: float) -> np.ndarray:
    """f of Eq. 6 and 8: layer normalisation over the last axis (biased variance, eps inside the root), then GeLU
    (the exact form, x Phi(x))."""
    from math import erf
    mu = x.mean(axis=-1, keepdims=True)
    var = ((x - mu) ** 2).mean(axis=-1, keepdims=True)
    y = (x - mu) / np.sqrt(var + eps)
    if gamma is not None:
        y = y * gamma
    if beta is not None:
        y = y + beta
    phi = 0.5 * (1.0 + np.vectorize(erf)(y / np.sqrt(2.0)))
    return y * phi


def lstm_cell(h_bits, emb_bits, w_bits, z, alpha: float, ln_c=(None, None), ln_z=(None, None), eps: float = 1e-5):
    """One step of the drafter cell, Eq. 1-8, in fp64.

    h_bits bf16 bits [M, d_in]: hidden states; emb_bits bf16 bits [M, d]: E(t), the embeddings of the tokens (Eq. 1);
    w_bits bf16 bits [4, d, d_in]: W^f, W^i, W^o, W^c stored output-major; z float [M, d]: the cell state (zeros at
    the first step).  Returns (h_next [M, d], z_next [M, d]):
        s^m = W^m h + alpha e                      (Eq. 2)
        g^m = sigmoid(s^m), m in {f, i, o}         (Eq. 5)
        s^c = f(s^c) g^i                           (Eq. 6)
        z   = z g^f + s^c                          (Eq. 7)
        h'  = f(z) g^o                             (Eq. 8)
    with f = layer normalisation followed by GeLU."""
    h = decode16(h_bits, "bf16").reshape(np.shape(h_bits))
    e = decode16(emb_bits, "bf16").reshape(np.shape(emb_bits))
    w = decode16(w_bits, "bf16").reshape(np.shape(w_bits))
    s = [h @ w[m].T + alpha * e for m in range(4)]
    sig = lambda x: 1.0 / (1.0 + np.exp(-x))
    gf, gi, go = sig(s[0]), sig(s[1]), sig(s[2])
    sc = _layer_norm_gelu(s[3], ln_c[0], ln_c[1], eps) * gi
    z_next = np.asarray(z, dtype=np.float64) * gf + sc
    h_next = _layer_norm_gelu(z_next, ln_z[0], ln_z[1], eps) * go
    return h_next, z_next

"""Thin ctypes binding of libowlverify (argument marshalling only; every step runs in the CUDA
kernels).  PyTorch supplies device memory and streams.  There is no fallback: if the shared
library has not been built, loading raises."""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libowlverify.so")
_lib = None

OWL_OK = 0
STATUS = {0: "OWL_OK", -1: "OWL_ERR_INVALID_ARG", -2: "OWL_ERR_UNSUPPORTED", -3: "OWL_ERR_CUDA",
          -4: "OWL_ERR_BAD_TREE", -5: "OWL_ERR_BAD_PAGE", -6: "OWL_ERR_TIMEOUT", -7: "OWL_ERR_TOO_LARGE"}


class OwlDims(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("total_nodes", ctypes.c_int32), ("max_nodes", ctypes.c_int32),
                ("num_q_heads", ctypes.c_int32), ("num_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
                ("page_size", ctypes.c_int32), ("max_pages_per_seq", ctypes.c_int32), ("num_pages", ctypes.c_int32),
                ("vocab", ctypes.c_int32), ("path_stride", ctypes.c_int32), ("sm_scale", ctypes.c_float)]


class OwlError(RuntimeError):
    def __init__(self, code: int, where: str, detail: str = ""):
        self.code = code
        super().__init__(f"{where}: {STATUS.get(code, code)} {detail}".strip())


def load_library() -> ctypes.CDLL:
    """dlopen the in-tree libowlverify.so; raises if it was not built (no CPU fallback exists)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2510_07535_b200.build` "
                          "(nvcc, sm_100a). There is no fallback path.")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64
    dp = ctypes.POINTER(OwlDims)
    lib.owl_create.restype = i32
    lib.owl_create.argtypes = [ctypes.POINTER(vp), i32, dp]
    lib.owl_destroy.restype = i32
    lib.owl_destroy.argtypes = [vp]
    lib.owl_verify_attn.restype = i32
    lib.owl_verify_attn.argtypes = [vp, dp] + [vp] * 10
    lib.owl_verify_attn_f16.restype = i32
    lib.owl_verify_attn_f16.argtypes = [vp, dp] + [vp] * 10
    lib.owl_tree_accept.restype = i32
    lib.owl_tree_accept.argtypes = [vp, dp] + [vp] * 9
    lib.owl_tree_accept_spec.restype = i32
    lib.owl_tree_accept_spec.argtypes = [vp, dp] + [vp] * 10
    lib.owl_prepare_spec_tree.restype = i32
    lib.owl_prepare_spec_tree.argtypes = [vp, dp] + [vp] * 4 + [ctypes.c_int32] + [vp] * 6
    lib.owl_prepare_hybrid.restype = i32
    lib.owl_prepare_hybrid.argtypes = [vp, dp] + [vp] * 5 + [ctypes.c_int32] + [vp] * 6
    lib.owl_howl_route.restype = i32
    lib.owl_howl_route.argtypes = [ctypes.c_int32, vp, ctypes.c_float, vp, vp]
    lib.owl_kv_commit.restype = i32
    lib.owl_kv_commit.argtypes = [vp, dp] + [vp] * 8
    lib.owl_lm_head_accept.restype = i32
    lib.owl_lm_head_accept.argtypes = [vp, dp, ctypes.c_int32] + [vp] * 10
    lib.owl_lstm_cell.restype = i32
    lib.owl_lstm_cell.argtypes = [vp, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, vp, vp, vp, ctypes.c_float, vp, vp, vp, vp,
                                  ctypes.c_float, vp, vp, vp, vp, vp]
    lib.owl_lstm_alpha.restype = ctypes.c_double
    lib.owl_lstm_alpha.argtypes = [ctypes.c_int32, ctypes.c_int32]
    lib.owl_tree_accept_static.restype = i32
    lib.owl_tree_accept_static.argtypes = [dp] + [vp] * 10
    lib.owl_verify_step.restype = i32
    lib.owl_verify_step.argtypes = [vp, dp] + [vp] * 16
    lib.owl_verify_step_host.restype = i32
    lib.owl_verify_step_host.argtypes = [vp, dp] + [vp] * 15
    lib.owl_get_status.restype = i32
    lib.owl_get_status.argtypes = [vp, vp]
    lib.owl_selftest_wait.restype = i32
    lib.owl_selftest_wait.argtypes = [vp, ctypes.c_uint64, ctypes.POINTER(ctypes.c_uint64), vp]
    lib.owl_status_string.restype = ctypes.c_char_p
    lib.owl_status_string.argtypes = [i32]
    lib.owl_last_error.restype = ctypes.c_char_p
    lib.owl_last_error.argtypes = [vp]
    lib.owl_launch_count.restype = i64
    lib.owl_launch_count.argtypes = [vp]
    lib.owl_set_profiling.restype = i32
    lib.owl_set_profiling.argtypes = [vp, i32]
    lib.owl_last_kernel_times.restype = i32
    lib.owl_last_kernel_times.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_double)]
    _lib = lib
    return lib


def _ptr(t: Optional[torch.Tensor], dtype: torch.dtype, device: torch.device, name: str):
    if t is None:
        return None
    if t.dtype != dtype or t.device != device or not t.is_contiguous():
        raise TypeError(f"{name}: expected contiguous {dtype} tensor on {device}, got {t.dtype} on {t.device}")
    return ctypes.c_void_p(t.data_ptr())


def _stream(device: torch.device) -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream(device).cuda_stream)


def make_dims(*, batch, total_nodes, max_nodes, num_q_heads=0, num_kv_heads=0, head_dim=128, page_size=16,
              max_pages_per_seq=0, num_pages=0, vocab=0, path_stride=64, sm_scale=1.0) -> OwlDims:
    return OwlDims(batch, total_nodes, max_nodes, num_q_heads, num_kv_heads, head_dim, page_size,
                   max_pages_per_seq, num_pages, vocab, path_stride, sm_scale)


class OwlContext:
    """Owner of one ``owl_ctx`` (device workspace).  Methods mirror the C entry points."""

    def __init__(self, max_dims: OwlDims, device: Optional[torch.device] = None):
        self.lib = load_library()
        self.device = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
        if self.device.index is None:
            self.device = torch.device("cuda", torch.cuda.current_device())
        self._h = ctypes.c_void_p()
        torch.cuda.init()
        rc = self.lib.owl_create(ctypes.byref(self._h), self.device.index, ctypes.byref(max_dims))
        if rc != OWL_OK:
            raise OwlError(rc, "owl_create")

    def close(self):
        if getattr(self, "_h", None) and self._h.value:
            torch.cuda.synchronize(self.device)
            self.lib.owl_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def owl_verify_attn(self, dims: OwlDims, q, k_cache, v_cache, block_table, ctx_lens, node_offsets, tree_parent,
                        out, lse, check: bool = True) -> int:
        dev = self.device
        rc = self.lib.owl_verify_attn(
            self._h, ctypes.byref(dims), _ptr(q, torch.bfloat16, dev, "q"), _ptr(k_cache, torch.bfloat16, dev, "k_cache"),
            _ptr(v_cache, torch.bfloat16, dev, "v_cache"), _ptr(block_table, torch.int32, dev, "block_table"),
            _ptr(ctx_lens, torch.int32, dev, "ctx_lens"), _ptr(node_offsets, torch.int32, dev, "node_offsets"),
            _ptr(tree_parent, torch.int32, dev, "tree_parent"), _ptr(out, torch.bfloat16, dev, "out"),
            _ptr(lse, torch.float32, dev, "lse"), _stream(dev))
        if check and rc != OWL_OK:
            raise OwlError(rc, "owl_verify_attn", self.last_error())
        return rc

    def owl_verify_attn_f16(self, dims: OwlDims, q, k_cache, v_cache, block_table, ctx_lens, node_offsets, tree_parent,
                            out, lse, check: bool = True) -> int:
        dev = self.device
        h = torch.float16
        rc = self.lib.owl_verify_attn_f16(
            self._h, ctypes.byref(dims), _ptr(q, h, dev, "q"), _ptr(k_cache, h, dev, "k_cache"), _ptr(v_cache, h, dev, "v_cache"),
            _ptr(block_table, torch.int32, dev, "block_table"), _ptr(ctx_lens, torch.int32, dev, "ctx_lens"),
            _ptr(node_offsets, torch.int32, dev, "node_offsets"), _ptr(tree_parent, torch.int32, dev, "tree_parent"),
            _ptr(out, h, dev, "out"), _ptr(lse, torch.float32, dev, "lse"), _stream(dev))
        if check and rc != OWL_OK:
            raise OwlError(rc, "owl_verify_attn_f16", self.last_error())
        return rc

    def owl_tree_accept(self, dims: OwlDims, logits, draft_tokens, node_offsets, tree_parent, accept_len, accept_path,
                        bonus_token, node_argmax=None, check: bool = True) -> int:
        dev = self.device
        rc = self.lib.owl_tree_accept(
            self._h, ctypes.byref(dims), _ptr(logits, torch.float32, dev, "logits"),
            _ptr(draft_tokens, torch.int32, dev, "draft_tokens"), _ptr(node_offsets, torch.int32, dev, "node_offsets"),
            _ptr(tree_parent, torch.int32, dev, "tree_parent"), _ptr(accept_len, torch.int32, dev, "accept_len"),
            _ptr(accept_path, torch.int32, dev, "accept_path"), _ptr(bonus_token, torch.int32, dev, "bonus_token"),
            _ptr(node_argmax, torch.int32, dev, "node_argmax"), _stream(dev))
        if check and rc != OWL_OK:
            raise OwlError(rc, "owl_tree_accept", self.last_error())
        return rc

    def owl_tree_accept_spec(self, dims: OwlDims, logits, draft_tokens, node_offsets, tree_parent, accept_len, accept_path,
                             bonus_token, spec_node, node_argmax=None, check: bool = True) -> int:
        dev = self.device
        i32 = torch.int32
        rc = self.lib.owl_tree_accept_spec(
            self._h, ctypes.byref(dims), _ptr(logits, torch.float32, dev, "logits"), _ptr(draft_tokens, i32, dev, "draft_tokens"),
            _ptr(node_offsets, i32, dev, "node_offsets"), _ptr(tree_parent, i32, dev, "tree_parent"),
            _ptr(accept_len, i32, dev, "accept_len"), _ptr(accept_path, i32, dev, "accept_path"),
            _ptr(bonus_token, i32, dev, "bonus_token"), _ptr(spec_node, i32, dev, "spec_node"),
            _ptr(node_argmax, i32, dev, "node_argmax"), _stream(dev))
        if check and rc != OWL_OK:
            raise OwlError(rc, "owl_tree_accept_spec", self.last_error())
        return rc

    def owl_prepare_spec_tree(self, dims: OwlDims, node_offsets, tree_parent, draft_tokens, ctx_lens, spec_token: int,
                              out_node_offsets, out_tree_parent, out_draft_tokens, out_input_ids, out_position_ids,
                              check: bool = True) -> int:
        dev = self.device
        i32 = torch.int32
        rc = self.lib.owl_prepare_spec_tree(
            self._h, ctypes.byref(dims), _ptr(node_offsets, i32, dev, "node_offsets"), _ptr(tree_parent, i32, dev, "tree_parent"),
            _ptr(draft_tokens, i32, dev, "draft_tokens"), _ptr(ctx_lens, i32, dev, "ctx_lens"), int(spec_token),
            _ptr(out_node_offsets, i32, dev, "out_node_offsets"), _ptr(out_tree_parent, i32, dev, "out_tree_parent"),
            _ptr(out_draft_tokens, i32, dev, "out_draft_tokens"), _ptr(out_input_ids, i32, dev, "out_input_ids"),
            _ptr(out_position_ids, i32, dev, "out_position_ids"), _stream(dev))
        if check and rc != OWL_OK:
            raise OwlError(rc, "owl_prepare_spec_tree", self.last_error())
        return rc

    def owl_prepare_hybrid(self, dims: OwlDims, node_offsets, tree_parent, draft_tokens, ctx_lens, route, spec_token: int,
                           out_node_offsets, out_tree_parent, out_draft_tokens, out_input_ids, out_position_ids,
                           check: bool = True) -> int:
        dev = self.device
        i32 = torch.int32
        rc = self.lib.owl_prepare_hybrid(
            self._h, ctypes.byref(dims), _ptr(node_offsets, i32, dev, "node_offsets"), _ptr(tree_parent, i32, dev, "tree_parent"),
            _ptr(draft_tokens, i32, dev, "draft_tokens"), _ptr(ctx_lens, i32, dev, "ctx_lens"), _ptr(route, i32, dev, "route"),
            int(spec_token), _ptr(out_node_offsets, i32, dev, "out_node_offsets"), _ptr(out_tree_parent, i32, dev, "out_tree_parent"),
            _ptr(out_draft_tokens, i32, dev, "out_draft_tokens"), _ptr(out_input_ids, i32, dev, "out_input_ids"),
            _ptr(out_position_ids, i32, dev, "out_position_ids"), _stream(dev))
        if check and rc != OWL_OK:
            raise OwlError(rc, "owl_prepare_hybrid", self.last_error())
        return rc

    def owl_kv_commit(self, dims: OwlDims, k_cache, v_cache, block_table, ctx_lens, node_offsets, accept_len, accept_path,
                      check: bool = True) -> int:
        dev = self.device
        i32, bf = torch.int32, torch.bfloat16
        rc = self.lib.owl_kv_commit(
            self._h, ctypes.byref(dims), _ptr(k_cache, bf, dev, "k_cache"), _ptr(v_cache, bf, dev, "v_cache"),
            _ptr(block_table, i32, dev, "block_table"), _ptr(ctx_lens, i32, dev, "ctx_lens"),
            _ptr(node_offsets, i32, dev, "node_offsets"), _ptr(accept_len, i32, dev, "accept_len"),
            _ptr(accept_path, i32, dev, "accept_path"), _stream(dev))
        if check and rc != OWL_OK:
            raise OwlError(rc, "owl_kv_commit", self.last_error())
        return rc

    def owl_lm_head_accept(self, dims: OwlDims, hidden, weight, draft_tokens, node_offsets, tree_parent, accept_len, accept_path,
                           bonus_token, node_argmax=None, check: bool = True) -> int:
        dev = self.device
        i32, bf = torch.int32, torch.bfloat16
        rc = self.lib.owl_lm_head_accept(
            self._h, ctypes.byref(dims), int((weight if hidden is None else hidden).shape[-1]), _ptr(hidden, bf, dev, "hidden"),
            _ptr(weight, bf, dev, "weight"),
            _ptr(draft_tokens, i32, dev, "draft_tokens"), _ptr(node_offsets, i32, dev, "node_offsets"),
            _ptr(tree_parent, i32, dev, "tree_parent"), _ptr(accept_len, i32, dev, "accept_len"),
            _ptr(accept_path, i32, dev, "accept_path"), _ptr(bonus_token, i32, dev, "bonus_token"),
            _ptr(node_argmax, i32, dev, "node_argmax"), _stream(dev))
        if check and rc != OWL_OK:
            raise OwlError(rc, "owl_lm_head_accept", self.last_error())
        return rc

    def owl_lstm_cell(self, h, emb, w, alpha: float, z, h_out_f32, h_out_bf16, workspace, ln_c=(None, None), ln_z=(None, None),
                      eps: float = 1e-5, check: bool = True) -> int:
        dev = self.device
        bf, f32 = torch.bfloat16, torch.float32
        rows, d_in = h.shape
        d = emb.shape[-1]
        rc = self.lib.owl_lstm_cell(
            self._h, rows, d_in, d, _ptr(h, bf, dev, "h"), _ptr(emb, bf, dev, "emb"), _ptr(w, bf, dev, "w"), float(alpha),
            _ptr(ln_c[0], f32, dev, "ln_c_gamma"), _ptr(ln_c[1], f32, dev, "ln_c_beta"), _ptr(ln_z[0], f32, dev, "ln_z_gamma"),
            _ptr(ln_z[1], f32, dev, "ln_z_beta"), float(eps), _ptr(z, f32, dev, "z"), _ptr(h_out_f32, f32, dev, "h_out_f32"),
            _ptr(h_out_bf16, bf, dev, "h_out_bf16"), _ptr(workspace, f32, dev, "workspace"), _stream(dev))
        if check and rc != OWL_OK:
            raise OwlError(rc, "owl_lstm_cell", self.last_error())
        return rc

    def owl_verify_step(self, dims: OwlDims, q, k_cache, v_cache, block_table, ctx_lens, node_offsets, tree_parent, out, lse,
                        logits, draft_tokens, accept_len, accept_path, bonus_token, node_argmax=None, check: bool = True) -> int:
        dev = self.device
        i32, bf, f32 = torch.int32, torch.bfloat16, torch.float32
        rc = self.lib.owl_verify_step(
            self._h, ctypes.byref(dims), _ptr(q, bf, dev, "q"), _ptr(k_cache, bf, dev, "k_cache"), _ptr(v_cache, bf, dev, "v_cache"),
            _ptr(block_table, i32, dev, "block_table"), _ptr(ctx_lens, i32, dev, "ctx_lens"),
            _ptr(node_offsets, i32, dev, "node_offsets"), _ptr(tree_parent, i32, dev, "tree_parent"), _ptr(out, bf, dev, "out"),
            _ptr(lse, f32, dev, "lse"), _ptr(logits, f32, dev, "logits"), _ptr(draft_tokens, i32, dev, "draft_tokens"),
            _ptr(accept_len, i32, dev, "accept_len"), _ptr(accept_path, i32, dev, "accept_path"),
            _ptr(bonus_token, i32, dev, "bonus_token"), _ptr(node_argmax, i32, dev, "node_argmax"), _stream(dev))
        if check and rc != OWL_OK:
            raise OwlError(rc, "owl_verify_step", self.last_error())
        return rc

    def owl_verify_step_host(self, dims: OwlDims, q, k_cache, v_cache, block_table, ctx_lens, node_offsets,
                             tree_parent, logits, draft_tokens, out, lse, accept_len, accept_path, bonus_token) -> int:
        """All tensors are HOST (CPU, ideally pinned) torch tensors; returns the device status word."""
        cpu = torch.device("cpu")
        args = [(q, torch.bfloat16), (k_cache, torch.bfloat16), (v_cache, torch.bfloat16), (block_table, torch.int32),
                (ctx_lens, torch.int32), (node_offsets, torch.int32), (tree_parent, torch.int32),
                (logits, torch.float32), (draft_tokens, torch.int32), (out, torch.bfloat16), (lse, torch.float32),
                (accept_len, torch.int32), (accept_path, torch.int32), (bonus_token, torch.int32)]
        ptrs = [_ptr(t, dt, cpu, f"arg{i}") for i, (t, dt) in enumerate(args)]
        rc = self.lib.owl_verify_step_host(self._h, ctypes.byref(dims), *ptrs, _stream(self.device))
        if rc in (-1, -2, -3, -7):
            raise OwlError(rc, "owl_verify_step_host", self.last_error())
        return rc

    def owl_get_status(self) -> int:
        return int(self.lib.owl_get_status(self._h, _stream(self.device)))

    def owl_selftest_wait(self, limit_ns: int):
        """Runs the kernels' bounded wait on a barrier nothing completes; returns (status, ns of the first wait,
        ns of the second wait)."""
        ns = (ctypes.c_uint64 * 2)()
        rc = int(self.lib.owl_selftest_wait(self._h, ctypes.c_uint64(limit_ns), ns, _stream(self.device)))
        return rc, int(ns[0]), int(ns[1])

    def last_error(self) -> str:
        return self.lib.owl_last_error(self._h).decode()

    def launch_count(self) -> int:
        return int(self.lib.owl_launch_count(self._h))

    def set_profiling(self, on: bool) -> None:
        self.lib.owl_set_profiling(self._h, 1 if on else 0)

    def last_kernel_times(self):
        t = (ctypes.c_double * 4)()
        rc = self.lib.owl_last_kernel_times(self._h, _stream(self.device), t)
        if rc != OWL_OK:
            raise OwlError(rc, "owl_last_kernel_times")
        return list(t)


STATIC_MAX_KEYS = 16384   # OWL_STATIC_MAX_KEYS of owlverify.h


def owl_tree_accept_static(dims: OwlDims, logits, draft_tokens, node_offsets, tree_parent, accept_len, accept_path,
                           bonus_token, node_argmax=None, device_status=None, check: bool = True) -> int:
    """Acceptance without a context and without any device allocation inside the library: for callers
    whose memory is managed elsewhere and who therefore cannot create an ``OwlContext``.  The tensors
    (allocated by the caller, as always) must live on the current CUDA device; scratch is the library's
    fixed array, shared by every call on that device, so overlapping calls must be serialised by the
    caller.  ``device_status`` (optional int32[1] on the device) receives 0 or OWL_ERR_BAD_TREE."""
    lib = load_library()
    dev = torch.device("cuda", torch.cuda.current_device())
    rc = lib.owl_tree_accept_static(
        ctypes.byref(dims), _ptr(logits, torch.float32, dev, "logits"),
        _ptr(draft_tokens, torch.int32, dev, "draft_tokens"), _ptr(node_offsets, torch.int32, dev, "node_offsets"),
        _ptr(tree_parent, torch.int32, dev, "tree_parent"), _ptr(accept_len, torch.int32, dev, "accept_len"),
        _ptr(accept_path, torch.int32, dev, "accept_path"), _ptr(bonus_token, torch.int32, dev, "bonus_token"),
        _ptr(node_argmax, torch.int32, dev, "node_argmax"), _ptr(device_status, torch.int32, dev, "device_status"),
        _stream(dev))
    if check and rc != OWL_OK:
        raise OwlError(rc, "owl_tree_accept_static")
    return rc


def owl_howl_route(score, c: float, lastwaslinear):
    """Algorithm 1's routing on HOST numpy arrays: score float32 [B]; lastwaslinear uint8 [B], updated in place.
    Returns route int32 [B] (0 linear, 1 tree from D_nospec, 2 tree from D_spec)."""
    import numpy as np
    lib = load_library()
    score = np.ascontiguousarray(score, dtype=np.float32)
    if lastwaslinear.dtype != np.uint8 or not lastwaslinear.flags["C_CONTIGUOUS"]:
        raise TypeError("lastwaslinear: contiguous uint8 array expected (it is updated in place)")
    route = np.empty(score.shape[0], np.int32)
    rc = lib.owl_howl_route(score.shape[0], score.ctypes.data_as(ctypes.c_void_p), float(c),
                            lastwaslinear.ctypes.data_as(ctypes.c_void_p), route.ctypes.data_as(ctypes.c_void_p))
    if rc != OWL_OK:
        raise OwlError(rc, "owl_howl_route")
    return route


def owl_lstm_alpha(n_depth: int, d: int) -> float:
    return float(load_library().owl_lstm_alpha(n_depth, d))


def status_string(code: int) -> str:
    return load_library().owl_status_string(code).decode()

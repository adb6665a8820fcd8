"""Thin ctypes binding of the C-ABI library (`include/lime.h`): argument marshalling only.

Functions carry the C entry points' names and take torch CUDA tensors (used purely as device memory) plus
plain integers; every step of the path runs inside the library's kernels.  There is no CPU fallback: if the
shared library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Dict, Optional, Sequence

import numpy as np
import torch

LIME_MAX_LAYERS = 16
LIME_F32, LIME_BF16 = 0, 1
LIME_PHI_SOFTMAX, LIME_PHI_SILU = 0, 1
_STATUS = {0: "LIME_OK", 1: "LIME_INVALID_ARG", 2: "LIME_UNSUPPORTED_SHAPE", 3: "LIME_WORKSPACE_TOO_SMALL",
           4: "LIME_CUDA_ERROR", 5: "LIME_NOT_READY", 6: "LIME_DEVICE_TIMEOUT", 7: "LIME_EXCEEDS_STATIC_SCRATCH"}

LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "liblime_b200.so")


class LimeError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str = ""):
        self.status = status
        super().__init__(f"{where}: {_STATUS.get(status, status)}" + (f" [{detail}]" if detail else ""))


class lime_config(ctypes.Structure):
    _fields_ = [("d", ctypes.c_int32), ("H", ctypes.c_int32), ("ell", ctypes.c_int32), ("n_layers", ctypes.c_int32),
                ("d_ff", ctypes.c_int32), ("dtype", ctypes.c_int32), ("phi", ctypes.c_int32), ("ln", ctypes.c_int32),
                ("gated_mlp", ctypes.c_int32), ("attn_scale", ctypes.c_float), ("cand_scale", ctypes.c_float),
                ("ln_eps", ctypes.c_float), ("cand_heads", ctypes.c_int32)]


_PtrArr = ctypes.c_void_p * LIME_MAX_LAYERS


class lime_weights(ctypes.Structure):
    _fields_ = [("links", ctypes.c_void_p), ("Wq", _PtrArr), ("Wk", _PtrArr), ("Wv", _PtrArr), ("Wg", _PtrArr),
                ("Wu", _PtrArr), ("Wo", _PtrArr), ("cand_Wq", ctypes.c_void_p), ("cand_Wk", ctypes.c_void_p),
                ("cand_Wv", ctypes.c_void_p)]


LIME_FFN_MAX_HIDDEN = 3


class lime_ffn(ctypes.Structure):
    _fields_ = [("n_hidden", ctypes.c_int32), ("widths", ctypes.c_int32 * LIME_FFN_MAX_HIDDEN),
                ("W", ctypes.c_void_p * (LIME_FFN_MAX_HIDDEN + 1)), ("b", ctypes.c_void_p * (LIME_FFN_MAX_HIDDEN + 1))]


EXPORTS = ("lime_create", "lime_destroy", "lime_set_weights", "lime_workspace_bytes", "lime_lengths_to_offsets",
           "lime_gather_history", "lime_gather_history_normalized", "lime_precompute_candidate_links", "lime_xor_layer",
           "lime_encode_user", "lime_encode_user_normalized",
           "lime_score_candidates", "lime_pack_corpus_cache", "lime_score_candidates_packed", "lime_set_context_mlp", "lime_contextualize_links", "lime_set_head",
           "lime_head_workspace_bytes", "lime_score_candidates_head", "lime_precompute_candidate_links_noalloc", "lime_device_status", "lime_selftest_wait_expiry", "lime_profile_start", "lime_profile_stop", "lime_last_cuda_error",
           "lime_version")

_lib_handle = None


def load_library(path: Optional[str] = None) -> ctypes.CDLL:
    """dlopen the C-ABI library and declare its prototypes. Raises if it has not been built."""
    global _lib_handle
    if _lib_handle is not None and path is None:
        return _lib_handle
    p = path or LIB_PATH
    if not os.path.exists(p):
        raise RuntimeError(f"{p} is missing: build it with `python -m paper_2510_18239_b200.build` "
                           "(there is no CPU fallback)")
    lib = ctypes.CDLL(p)
    vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
    lib.lime_create.argtypes = [ctypes.POINTER(lime_config), ctypes.POINTER(vp)]
    lib.lime_destroy.argtypes = [vp]
    lib.lime_set_weights.argtypes = [vp, ctypes.POINTER(lime_weights), vp]
    lib.lime_workspace_bytes.argtypes = [vp, i32, i64]
    lib.lime_workspace_bytes.restype = sz
    lib.lime_lengths_to_offsets.argtypes = [vp, vp, i32, vp, vp]
    lib.lime_gather_history.argtypes = [vp, vp, i64, vp, i64, vp, vp, vp]
    lib.lime_gather_history_normalized.argtypes = [vp, vp, i64, vp, i64, vp, vp, vp]
    lib.lime_precompute_candidate_links.argtypes = [vp, vp, i64, vp, vp]
    lib.lime_xor_layer.argtypes = [vp, i32, vp, vp, i32, i64, vp, i32, vp, vp, vp, sz, vp]
    lib.lime_encode_user.argtypes = [vp, vp, vp, i32, i64, vp, vp, vp, sz, vp]
    lib.lime_encode_user_normalized.argtypes = [vp, vp, vp, i32, i64, vp, vp, vp, sz, vp]
    lib.lime_score_candidates.argtypes = [vp, vp, i32, vp, vp, vp, i32, i64, vp, i64, vp, vp, vp]
    lib.lime_pack_corpus_cache.argtypes = [vp, vp, vp, i64, vp, vp]
    lib.lime_score_candidates_packed.argtypes = [vp, vp, i32, vp, i64, vp, vp, i32, i64, vp, vp, vp]
    lib.lime_set_context_mlp.argtypes = [vp, i32, ctypes.POINTER(lime_ffn), vp]
    lib.lime_contextualize_links.argtypes = [vp, vp, i32, vp, vp]
    lib.lime_set_head.argtypes = [vp, ctypes.POINTER(lime_ffn), vp]
    lib.lime_head_workspace_bytes.argtypes = [vp, i32]
    lib.lime_head_workspace_bytes.restype = sz
    lib.lime_score_candidates_head.argtypes = [vp, vp, i32, vp, vp, vp, i32, i64, vp, i64, vp, vp, vp, sz, vp]
    lib.lime_precompute_candidate_links_noalloc.argtypes = [i32, i32, i32, ctypes.c_float, vp, vp, vp, vp, i64, vp, vp]
    lib.lime_device_status.argtypes = [vp, ctypes.POINTER(i32)]
    lib.lime_selftest_wait_expiry.argtypes = [vp, i32, vp]
    lib.lime_profile_start.argtypes = [i32]
    lib.lime_profile_stop.argtypes = [ctypes.c_char_p, sz, ctypes.POINTER(ctypes.c_float), i32, ctypes.POINTER(i32)]
    for name in EXPORTS:
        fn = getattr(lib, name)
        if name in ("lime_last_cuda_error", "lime_version"):
            fn.restype = ctypes.c_char_p
            fn.argtypes = []
        elif name not in ("lime_workspace_bytes", "lime_head_workspace_bytes"):
            fn.restype = ctypes.c_int
    if path is None:
        _lib_handle = lib
    return lib


def _check(status: int, where: str):
    if status != 0:
        detail = load_library().lime_last_cuda_error().decode() if status == 4 else ""
        raise LimeError(status, where, detail)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


# ----------------------------------------------------------------------------- 1:1 entry points
def lime_version() -> str:
    return load_library().lime_version().decode()


def lime_create(cfg: lime_config) -> int:
    h = ctypes.c_void_p()
    _check(load_library().lime_create(ctypes.byref(cfg), ctypes.byref(h)), "lime_create")
    return h.value


def lime_destroy(ctx: int) -> None:
    _check(load_library().lime_destroy(ctx), "lime_destroy")


def lime_set_weights(ctx: int, w: lime_weights) -> None:
    _check(load_library().lime_set_weights(ctx, ctypes.byref(w), _stream()), "lime_set_weights")


def lime_workspace_bytes(ctx: int, B: int, total_tokens: int) -> int:
    return int(load_library().lime_workspace_bytes(ctx, B, total_tokens))


def lime_lengths_to_offsets(ctx: int, lengths: torch.Tensor, off: torch.Tensor) -> None:
    _check(load_library().lime_lengths_to_offsets(ctx, _ptr(lengths), lengths.numel(), _ptr(off), _stream()),
           "lime_lengths_to_offsets")


def lime_gather_history(ctx: int, table: torch.Tensor, ids: torch.Tensor, out: torch.Tensor,
                        dev_flag: Optional[torch.Tensor] = None) -> None:
    _check(load_library().lime_gather_history(ctx, _ptr(table), table.shape[0], _ptr(ids), ids.numel(), _ptr(out),
                                              _ptr(dev_flag), _stream()), "lime_gather_history")


def lime_gather_history_normalized(ctx: int, table: torch.Tensor, ids: torch.Tensor, out: torch.Tensor,
                                   dev_flag: Optional[torch.Tensor] = None) -> None:
    _check(load_library().lime_gather_history_normalized(ctx, _ptr(table), table.shape[0], _ptr(ids), ids.numel(), _ptr(out),
                                                         _ptr(dev_flag), _stream()), "lime_gather_history_normalized")


def lime_precompute_candidate_links(ctx: int, cand_emb: torch.Tensor, out_w: torch.Tensor) -> None:
    _check(load_library().lime_precompute_candidate_links(ctx, _ptr(cand_emb), cand_emb.shape[0], _ptr(out_w), _stream()),
           "lime_precompute_candidate_links")


def lime_xor_layer(ctx: int, layer: int, hist_in: torch.Tensor, off: torch.Tensor, B: int, links_in: torch.Tensor,
                   links_shared: bool, hist_out: Optional[torch.Tensor], links_out: torch.Tensor,
                   ws: torch.Tensor) -> None:
    _check(load_library().lime_xor_layer(ctx, layer, _ptr(hist_in), _ptr(off), B, hist_in.shape[0], _ptr(links_in),
                                         1 if links_shared else 0, _ptr(hist_out), _ptr(links_out), _ptr(ws),
                                         ws.numel() * ws.element_size(), _stream()), "lime_xor_layer")


def lime_encode_user(ctx: int, hist: torch.Tensor, off: torch.Tensor, B: int, link_ctx: Optional[torch.Tensor],
                     link_states: torch.Tensor, ws: torch.Tensor) -> None:
    _check(load_library().lime_encode_user(ctx, _ptr(hist), _ptr(off), B, hist.shape[0], _ptr(link_ctx),
                                           _ptr(link_states), _ptr(ws), ws.numel() * ws.element_size(), _stream()),
           "lime_encode_user")


def lime_encode_user_normalized(ctx: int, hist_normalized: torch.Tensor, off: torch.Tensor, B: int,
                                link_ctx: Optional[torch.Tensor], link_states: torch.Tensor, ws: torch.Tensor) -> None:
    _check(load_library().lime_encode_user_normalized(ctx, _ptr(hist_normalized), _ptr(off), B, hist_normalized.shape[0],
                                                      _ptr(link_ctx), _ptr(link_states), _ptr(ws),
                                                      ws.numel() * ws.element_size(), _stream()),
           "lime_encode_user_normalized")


def lime_score_candidates(ctx: int, link_states: torch.Tensor, B: int, cand_w: torch.Tensor, cand_emb: torch.Tensor,
                          cand_off: Optional[torch.Tensor], C: int, total_cands: int,
                          cand_ids: Optional[torch.Tensor], logits: torch.Tensor, corpus_rows: Optional[int] = None,
                          dev_flag: Optional[torch.Tensor] = None) -> None:
    """corpus_rows (only with cand_ids): rows of the corpus caches cand_w / cand_emb; by default the row count of cand_emb."""
    if cand_ids is not None and corpus_rows is None:
        corpus_rows = int(cand_emb.shape[0])
    _check(load_library().lime_score_candidates(ctx, _ptr(link_states), B, _ptr(cand_w), _ptr(cand_emb), _ptr(cand_off),
                                                C, total_cands, _ptr(cand_ids), int(corpus_rows or 0), _ptr(dev_flag),
                                                _ptr(logits), _stream()),
           "lime_score_candidates")


def lime_pack_corpus_cache(ctx: int, cand_emb: torch.Tensor, cand_w: torch.Tensor, packed: torch.Tensor) -> None:
    _check(load_library().lime_pack_corpus_cache(ctx, _ptr(cand_emb), _ptr(cand_w), cand_emb.shape[0], _ptr(packed), _stream()),
           "lime_pack_corpus_cache")


def lime_score_candidates_packed(ctx: int, link_states: torch.Tensor, B: int, packed: torch.Tensor, cand_ids: torch.Tensor,
                                 cand_off: Optional[torch.Tensor], C: int, total_cands: int, logits: torch.Tensor,
                                 dev_flag: Optional[torch.Tensor] = None) -> None:
    _check(load_library().lime_score_candidates_packed(ctx, _ptr(link_states), B, _ptr(packed), packed.shape[0], _ptr(cand_ids),
                                                       _ptr(cand_off), C, total_cands, _ptr(dev_flag), _ptr(logits), _stream()),
           "lime_score_candidates_packed")


def make_ffn(layers) -> lime_ffn:
    """layers: list of (W tensor [in x out], b fp32 tensor [out] or None); all but the last are hidden layers."""
    f = lime_ffn()
    f.n_hidden = len(layers) - 1
    for i, (W, b) in enumerate(layers):
        if i < len(layers) - 1:
            f.widths[i] = int(W.shape[1])
        f.W[i] = _ptr(W)
        f.b[i] = _ptr(b)
    return f


def lime_set_context_mlp(ctx: int, d_c: int, mlp: lime_ffn) -> None:
    _check(load_library().lime_set_context_mlp(ctx, d_c, ctypes.byref(mlp), _stream()), "lime_set_context_mlp")


def lime_contextualize_links(ctx: int, user_ctx: torch.Tensor, B: int, link_ctx: torch.Tensor) -> None:
    _check(load_library().lime_contextualize_links(ctx, _ptr(user_ctx), B, _ptr(link_ctx), _stream()), "lime_contextualize_links")


def lime_set_head(ctx: int, head: lime_ffn) -> None:
    _check(load_library().lime_set_head(ctx, ctypes.byref(head), _stream()), "lime_set_head")


def lime_head_workspace_bytes(ctx: int, B: int) -> int:
    return int(load_library().lime_head_workspace_bytes(ctx, B))


def lime_score_candidates_head(ctx: int, link_states: torch.Tensor, B: int, cand_w: torch.Tensor, cand_emb: torch.Tensor,
                               cand_off: Optional[torch.Tensor], C: int, total_cands: int, cand_ids: Optional[torch.Tensor],
                               logits: torch.Tensor, ws: torch.Tensor, corpus_rows: Optional[int] = None,
                               dev_flag: Optional[torch.Tensor] = None) -> None:
    if cand_ids is not None and corpus_rows is None:
        corpus_rows = int(cand_emb.shape[0])
    _check(load_library().lime_score_candidates_head(ctx, _ptr(link_states), B, _ptr(cand_w), _ptr(cand_emb), _ptr(cand_off),
                                                     C, total_cands, _ptr(cand_ids), int(corpus_rows or 0), _ptr(dev_flag),
                                                     _ptr(logits), _ptr(ws), ws.numel() * ws.element_size(), _stream()),
           "lime_score_candidates_head")


def lime_precompute_candidate_links_noalloc(dtype: int, d: int, ell: int, cand_scale: float, links: torch.Tensor,
                                            cand_Wq: Optional[torch.Tensor], cand_Wk: Optional[torch.Tensor],
                                            cand_emb: torch.Tensor, out_w: torch.Tensor) -> None:
    """Context-free, allocation-free precompute for callers that may not allocate device memory; the caller passes
    every buffer, including the output.  Raises LimeError(LIME_EXCEEDS_STATIC_SCRATCH) if ell * d is too large."""
    st = load_library().lime_precompute_candidate_links_noalloc(dtype, d, ell, cand_scale, _ptr(links), _ptr(cand_Wq),
                                                                _ptr(cand_Wk), _ptr(cand_emb), cand_emb.shape[0],
                                                                _ptr(out_w), _stream())
    if st != 0:
        raise LimeError(st, "lime_precompute_candidate_links_noalloc",
                        load_library().lime_last_cuda_error().decode() if st in (4, 7) else "")


def lime_device_status(ctx: int) -> int:
    """Synchronises; raises LimeError(LIME_DEVICE_TIMEOUT) if a bounded in-kernel wait gave up, else returns 0."""
    code = ctypes.c_int32(0)
    st = load_library().lime_device_status(ctx, ctypes.byref(code))
    if st != 0:
        raise LimeError(st, "lime_device_status", f"wait code {code.value}")
    return int(code.value)


def lime_selftest_wait_expiry(ctx: int, limit_us: int) -> None:
    """Launches a wait that can never be satisfied, bounded by limit_us; lime_device_status then reports the time-out."""
    _check(load_library().lime_selftest_wait_expiry(ctx, limit_us, _stream()), "lime_selftest_wait_expiry")


def lime_profile_start(capacity: int = 4096) -> None:
    _check(load_library().lime_profile_start(capacity), "lime_profile_start")


def lime_profile_stop(capacity: int = 4096):
    """Returns (list of (kernel name, milliseconds) in launch order, number of launches seen)."""
    names = ctypes.create_string_buffer(64 * capacity)
    ms = (ctypes.c_float * capacity)()
    count = ctypes.c_int32(0)
    _check(load_library().lime_profile_stop(names, len(names), ms, capacity, ctypes.byref(count)), "lime_profile_stop")
    nm = names.value.decode().split("\n")[:-1]
    return [(nm[i], float(ms[i])) for i in range(min(len(nm), count.value, capacity))], int(count.value)


# ----------------------------------------------------------------------------- storage <-> torch
def to_device(arr: np.ndarray, dtype: str, device="cuda") -> torch.Tensor:
    """A stored numpy array (fp32, uint16 bf16 bit patterns, or int32) as a CUDA tensor of the matching type."""
    if arr.dtype == np.uint16:
        return torch.from_numpy(arr.view(np.int16)).to(device).view(torch.bfloat16)
    return torch.from_numpy(np.ascontiguousarray(arr)).to(device)


def torch_dtype(dtype: int):
    return torch.float32 if dtype == LIME_F32 else torch.bfloat16


# ----------------------------------------------------------------------------- convenience wrapper
class Lime:
    """Owns a library context and the device buffers a caller would otherwise juggle by hand."""

    def __init__(self, d: int, H: int, ell: int, n_layers: int, dtype: int = LIME_BF16, d_ff: int = 0,
                 phi: int = LIME_PHI_SOFTMAX, ln: bool = True, gated_mlp: bool = True, attn_scale: float = 0.0,
                 cand_scale: float = 0.0, ln_eps: float = 0.0, cand_heads: int = 0):
        self.cfg = lime_config(d, H, ell, n_layers, d_ff, dtype, phi, int(ln), int(gated_mlp), attn_scale, cand_scale, ln_eps,
                               cand_heads)
        self.ell_c = ell * (H if cand_heads == H and H > 1 else 1)      # weight columns per candidate, link-state rows
        self.ctx = lime_create(self.cfg)
        self.tdtype = torch_dtype(dtype)
        self._keep = []
        self._ws = None

    def close(self):
        if self.ctx:
            lime_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_weights(self, links: torch.Tensor, layers: Sequence[Dict[str, Optional[torch.Tensor]]],
                    cand: Optional[Dict[str, torch.Tensor]] = None) -> None:
        w = lime_weights()
        w.links = _ptr(links)
        keep = [links]
        for j, lw in enumerate(layers):
            for name in ("Wq", "Wk", "Wv", "Wg", "Wu", "Wo"):
                t = lw.get(name)
                if t is not None:
                    getattr(w, name)[j] = _ptr(t)
                    keep.append(t)
        for name in ("Wq", "Wk", "Wv"):
            t = (cand or {}).get(name)
            if t is not None:
                setattr(w, "cand_" + name, _ptr(t))
                keep.append(t)
        lime_set_weights(self.ctx, w)
        self._keep = keep

    def workspace(self, B: int, total_tokens: int) -> torch.Tensor:
        need = lime_workspace_bytes(self.ctx, B, total_tokens)
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.empty(need, dtype=torch.uint8, device="cuda")
        return self._ws

    def lengths_to_offsets(self, lengths: torch.Tensor) -> torch.Tensor:
        off = torch.empty(lengths.numel() + 1, dtype=torch.int32, device=lengths.device)
        lime_lengths_to_offsets(self.ctx, lengths, off)
        return off

    def gather_history(self, table: torch.Tensor, ids: torch.Tensor, flag: Optional[torch.Tensor] = None) -> torch.Tensor:
        out = torch.empty((ids.numel(), self.cfg.d), dtype=self.tdtype, device=ids.device)
        lime_gather_history(self.ctx, table, ids, out, flag)
        return out

    def gather_history_normalized(self, table: torch.Tensor, ids: torch.Tensor,
                                  flag: Optional[torch.Tensor] = None) -> torch.Tensor:
        out = torch.empty((ids.numel(), self.cfg.d), dtype=self.tdtype, device=ids.device)
        lime_gather_history_normalized(self.ctx, table, ids, out, flag)
        return out

    def encode_user_normalized(self, hist_normalized: torch.Tensor, off: torch.Tensor,
                               link_ctx: Optional[torch.Tensor] = None) -> torch.Tensor:
        B = off.numel() - 1
        ls = torch.empty((B, self.ell_c, self.cfg.d), dtype=self.tdtype, device=hist_normalized.device)
        lime_encode_user_normalized(self.ctx, hist_normalized, off, B, link_ctx, ls, self.workspace(B, hist_normalized.shape[0]))
        return ls

    def precompute_candidate_links(self, cand_emb: torch.Tensor) -> torch.Tensor:
        out = torch.empty((cand_emb.shape[0], self.ell_c), dtype=self.tdtype, device=cand_emb.device)
        lime_precompute_candidate_links(self.ctx, cand_emb, out)
        return out

    def encode_user(self, hist: torch.Tensor, off: torch.Tensor, link_ctx: Optional[torch.Tensor] = None) -> torch.Tensor:
        B = off.numel() - 1
        ls = torch.empty((B, self.ell_c, self.cfg.d), dtype=self.tdtype, device=hist.device)
        lime_encode_user(self.ctx, hist, off, B, link_ctx, ls, self.workspace(B, hist.shape[0]))
        return ls

    def score_candidates(self, link_states: torch.Tensor, cand_w: torch.Tensor, cand_emb: torch.Tensor, C: int = 0,
                         cand_off: Optional[torch.Tensor] = None, cand_ids: Optional[torch.Tensor] = None,
                         total_cands: Optional[int] = None, corpus_rows: Optional[int] = None,
                         dev_flag: Optional[torch.Tensor] = None) -> torch.Tensor:
        B = link_states.shape[0]
        total = total_cands if total_cands is not None else (cand_ids.numel() if cand_ids is not None else cand_emb.shape[0])
        logits = torch.empty(total, dtype=torch.float32, device=link_states.device)
        lime_score_candidates(self.ctx, link_states, B, cand_w, cand_emb, cand_off, C, total, cand_ids, logits, corpus_rows, dev_flag)
        return logits

    def pack_corpus_cache(self, cand_emb: torch.Tensor, cand_w: torch.Tensor) -> torch.Tensor:
        packed = torch.empty((cand_emb.shape[0], self.cfg.d + self.ell_c), dtype=self.tdtype, device=cand_emb.device)
        lime_pack_corpus_cache(self.ctx, cand_emb, cand_w, packed)
        return packed

    def score_candidates_packed(self, link_states: torch.Tensor, packed: torch.Tensor, cand_ids: torch.Tensor, C: int = 0,
                                cand_off: Optional[torch.Tensor] = None, dev_flag: Optional[torch.Tensor] = None) -> torch.Tensor:
        logits = torch.empty(cand_ids.numel(), dtype=torch.float32, device=link_states.device)
        lime_score_candidates_packed(self.ctx, link_states, link_states.shape[0], packed, cand_ids, cand_off, C, cand_ids.numel(),
                                     logits, dev_flag)
        return logits

    # ---- feed-forward networks (Eq. 2; the interaction network of Sec. 3.3)
    def set_context_mlp(self, d_c: int, layers) -> None:
        self._keep_ctx = [t for pair in layers for t in pair if t is not None]
        lime_set_context_mlp(self.ctx, d_c, make_ffn(layers))

    def contextualize_links(self, user_ctx: torch.Tensor) -> torch.Tensor:
        B = user_ctx.shape[0]
        out = torch.empty((B, self.cfg.ell, self.cfg.d), dtype=torch.float32, device=user_ctx.device)
        lime_contextualize_links(self.ctx, user_ctx, B, out)
        return out

    def set_head(self, layers) -> None:
        self._keep_head = [t for pair in layers for t in pair if t is not None]
        lime_set_head(self.ctx, make_ffn(layers))

    def score_candidates_head(self, link_states: torch.Tensor, cand_w: torch.Tensor, cand_emb: torch.Tensor, C: int = 0,
                              cand_off: Optional[torch.Tensor] = None, cand_ids: Optional[torch.Tensor] = None,
                              total_cands: Optional[int] = None, corpus_rows: Optional[int] = None,
                              dev_flag: Optional[torch.Tensor] = None) -> torch.Tensor:
        B = link_states.shape[0]
        total = total_cands if total_cands is not None else (cand_ids.numel() if cand_ids is not None else cand_emb.shape[0])
        logits = torch.empty(total, dtype=torch.float32, device=link_states.device)
        need = lime_head_workspace_bytes(self.ctx, B)
        if getattr(self, "_head_ws", None) is None or self._head_ws.numel() < need:
            self._head_ws = torch.empty(need, dtype=torch.uint8, device=link_states.device)
        lime_score_candidates_head(self.ctx, link_states, B, cand_w, cand_emb, cand_off, C, total, cand_ids, logits,
                                   self._head_ws, corpus_rows, dev_flag)
        return logits

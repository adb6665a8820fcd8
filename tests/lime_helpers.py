"""Glue used by the parity tests: the same seeded stored arrays go to the fp64 oracle (widened) and to the
CUDA library (as device tensors).  No arithmetic of the method lives here."""
from __future__ import annotations

from typing import Dict, List, Optional

import numpy as np

from oracle import lime_oracle as O
from paper_2510_18239_b200 import synth

LAYER_KEYS = ("Wq", "Wk", "Wv", "Wg", "Wu", "Wo")


def oracle_config(wl: synth.Workload, phi=O.SOFTMAX, ln=True, gated_mlp=True, attn_scale=None) -> O.OracleConfig:
    return O.OracleConfig(d=wl.d, H=wl.H, ell=wl.ell, n_layers=wl.n_layers, phi=phi, ln=ln, gated_mlp=gated_mlp,
                          attn_scale=attn_scale)


def oracle_layers(inp: Dict[str, np.ndarray], wl: synth.Workload, gated_mlp=True) -> List[Dict[str, np.ndarray]]:
    layers = []
    for j in range(wl.n_layers):
        lw = {k: synth.storage_to_f64(inp[k][j], wl.dtype) for k in LAYER_KEYS}
        if not gated_mlp:
            for k in ("Wg", "Wu", "Wo"):
                lw.pop(k)
        layers.append(lw)
    return layers


def oracle_user(inp, wl, b: int, off: np.ndarray, table64: np.ndarray, links64: np.ndarray, layers, cfg,
                cand_rows: Optional[np.ndarray] = None, cand_w=None, cand_heads: bool = False, head=None, LC=None):
    """Oracle logits / link states / weights for user b (optionally only candidate slots `cand_rows` of that user)."""
    E = O.gather_history(table64, inp["hist_ids"][off[b]:off[b + 1]])
    cids = inp["cand_ids"][b * wl.C:(b + 1) * wl.C]
    if cand_rows is not None:
        cids = cids[cand_rows]
    T = O.gather_history(table64, cids)
    return O.run_user(E, links64, layers, cfg, T, LC=LC, cand_w=cand_w, cand_heads=cand_heads, head=head)


class LazyTable64:
    """The stored embedding table seen as fp64 rows, widened row by row on demand (the largest table is 4M x 256:
    widening all of it would take 8 GB); indexable the way the oracle's lookup indexes a table."""

    def __init__(self, table: np.ndarray, dtype: str):
        self._table, self._dtype, self._rows = table, dtype, {}
        self.shape, self.dtype = table.shape, np.float64

    def __getitem__(self, key):
        i = int(key[0] if isinstance(key, tuple) else key)
        r = self._rows.get(i)
        if r is None:
            r = synth.storage_to_f64(self._table[i], self._dtype)
            self._rows[i] = r
        return r


class DeviceBatch:
    """Device-side mirror of one synthetic batch plus a configured library context."""

    def __init__(self, wl: synth.Workload, inp: Dict[str, np.ndarray], phi=0, ln=True, gated_mlp=True, cand=None,
                 attn_scale=0.0, cand_heads=0):
        import torch
        from paper_2510_18239_b200 import binding as Bd
        self.Bd = Bd
        self.wl = wl
        dt = Bd.LIME_F32 if wl.dtype == synth.F32 else Bd.LIME_BF16
        self.lime = Bd.Lime(wl.d, wl.H, wl.ell, wl.n_layers, dtype=dt, d_ff=wl.d_ff, phi=phi, ln=ln, gated_mlp=gated_mlp,
                            attn_scale=attn_scale, cand_heads=cand_heads)
        self.table = Bd.to_device(inp["table"], wl.dtype)
        self.links = Bd.to_device(inp["links"], wl.dtype)
        self.w = {k: Bd.to_device(inp[k], wl.dtype) for k in LAYER_KEYS}
        layers = [{k: self.w[k][j] for k in LAYER_KEYS} for j in range(wl.n_layers)]
        self.cand = {k: Bd.to_device(v, wl.dtype) for k, v in (cand or {}).items()}
        self.lime.set_weights(self.links, layers, self.cand)
        self.lengths = torch.from_numpy(inp["lengths"]).cuda()
        self.hist_ids = torch.from_numpy(inp["hist_ids"]).cuda()
        self.cand_ids = torch.from_numpy(inp["cand_ids"]).cuda() if "cand_ids" in inp else None

    def run(self, normalized=False):
        """offsets -> gather -> encode -> (candidate gather, precompute) -> score. Returns dict of tensors.
        normalized: take the history through the fused lookup + LayerNorm and the encode entry that expects it."""
        L = self.lime
        off = L.lengths_to_offsets(self.lengths)
        if normalized:
            hist = L.gather_history_normalized(self.table, self.hist_ids)
            ls = L.encode_user_normalized(hist, off)
        else:
            hist = L.gather_history(self.table, self.hist_ids)
            ls = L.encode_user(hist, off)
        cand = L.gather_history(self.table, self.cand_ids)
        W = L.precompute_candidate_links(cand)
        logits = L.score_candidates(ls, W, cand, C=self.wl.C)
        self.Bd.lime_device_status(L.ctx)      # synchronises; raises if a bounded in-kernel wait gave up
        return dict(off=off, hist=hist, link_states=ls, cand=cand, W=W, logits=logits)


def to_f64(t) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)

"""Seeded synthetic inputs for LIME ranking inference workloads.

This module only *draws* inputs (embedding tables, link embeddings, projection
weights, ragged history lengths, Zipf-skewed history ids, candidate ids) and
converts between storage formats (fp32 <-> bf16 bit patterns).  It contains
none of the method's arithmetic, so both the CPU oracle's tests and the CUDA
path's tests may feed from it without sharing any computation.

Workload shapes follow the paper's synthetic latency study (sweeps over the
number of candidates and the history length, App. F) and its hyper-parameter
table (H = 4 heads, 8..32 links, histories up to 1024; App. C), scaled up as the
five named workloads below.

Every array is a pure function of (workload, seed, stream name): each stream has
its own counter-based Philox generator keyed by the seed and a per-stream tag,
so the order in which streams are drawn does not matter.
"""
from __future__ import annotations

import dataclasses
import zlib
from typing import Dict, Optional, Tuple

import numpy as np

F32 = "f32"
BF16 = "bf16"


# --------------------------------------------------------------------------- #
# storage formats
# --------------------------------------------------------------------------- #
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (round-to-nearest-even); returns the uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = (u + np.uint32(0x7FFF) + lsb) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns (uint16) to the fp32 values they denote (exact)."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def to_storage(x: np.ndarray, dtype: str) -> np.ndarray:
    """fp32/fp64 values -> the array as it is stored for `dtype` (fp32 array, or bf16 bits)."""
    x32 = np.ascontiguousarray(x, dtype=np.float32)
    return x32 if dtype == F32 else f32_to_bf16_bits(x32)


def storage_to_f64(x: np.ndarray, dtype: str) -> np.ndarray:
    """Stored array -> the exact values it denotes, widened to fp64."""
    if dtype == F32:
        return np.asarray(x, dtype=np.float32).astype(np.float64)
    return bf16_bits_to_f32(x).astype(np.float64)


# --------------------------------------------------------------------------- #
# workloads
# --------------------------------------------------------------------------- #
@dataclasses.dataclass(frozen=True)
class Workload:
    """Shape of one batch of ranking requests (the paper's notation in brackets)."""

    name: str
    B: int                      # users in the batch
    n_min: int                  # shortest history [N(U)]
    n_max: int                  # longest history; n_min == n_max => dense batch
    d: int                      # embedding dimension [d]
    H: int                      # attention heads
    ell: int                    # link embeddings [l]
    n_layers: int               # stacked XOR layers [n]
    C: int                      # candidates per user [M(U)]
    dtype: str                  # storage type of activations / weights
    V: int                      # rows of the embedding table
    zipf_s: Optional[float]     # history-id skew; None => every id used once (i.i.d. rows)
    table_std: float            # std of table entries
    link_std: float             # std of link embeddings
    d_ff: int = 0               # GatedMLP width (0 => d)

    @property
    def dff(self) -> int:
        return self.d_ff or self.d

    @property
    def ragged(self) -> bool:
        return self.n_min != self.n_max

    def replace(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


def named_workloads() -> Dict[str, Workload]:
    """The five benchmark workloads (candidate and history sweeps take `.replace(C=..)` / `(n_min=..,n_max=..)`)."""
    w = {}
    # tiny fp32: all embeddings i.i.d. with variance 1/d; the table holds exactly one row per use.
    w["tiny_fp32"] = Workload("tiny_fp32", B=4, n_min=64, n_max=64, d=64, H=2, ell=8, n_layers=1, C=128,
                              dtype=F32, V=4 * 64 + 4 * 128, zipf_s=None, table_std=64 ** -0.5,
                              link_std=64 ** -0.5)
    w["bf16_baseline"] = Workload("bf16_baseline", B=256, n_min=512, n_max=512, d=128, H=4, ell=32,
                                  n_layers=2, C=2048, dtype=BF16, V=1_000_000, zipf_s=1.1,
                                  table_std=0.02, link_std=1.0)
    w["candidate_sweep"] = Workload("candidate_sweep", B=64, n_min=1024, n_max=1024, d=128, H=4, ell=32,
                                    n_layers=2, C=32768, dtype=BF16, V=1_000_000, zipf_s=1.1,
                                    table_std=0.02, link_std=1.0)
    w["long_history"] = Workload("long_history", B=32, n_min=32768, n_max=32768, d=128, H=4, ell=64,
                                 n_layers=4, C=1024, dtype=BF16, V=1_000_000, zipf_s=1.1,
                                 table_std=0.02, link_std=1.0)
    w["production_ragged"] = Workload("production_ragged", B=1024, n_min=1024, n_max=4096, d=256, H=8,
                                      ell=64, n_layers=4, C=8192, dtype=BF16, V=4_000_000, zipf_s=1.05,
                                      table_std=0.02, link_std=1.0)
    return w


CANDIDATE_SWEEP_C = tuple(2 ** k for k in range(4, 16))       # 16 .. 32768
LONG_HISTORY_N = tuple(2 ** k for k in range(10, 16))         # 1024 .. 32768


# --------------------------------------------------------------------------- #
# generators
# --------------------------------------------------------------------------- #
def _rng(seed: int, stream: str) -> np.random.Generator:
    tag = zlib.crc32(stream.encode("utf-8"))
    return np.random.Generator(np.random.Philox(np.random.SeedSequence([int(seed), int(tag)])))


def normal_storage(seed: int, stream: str, shape: Tuple[int, ...], std: float, dtype: str,
                   chunk_rows: int = 1 << 18) -> np.ndarray:
    """i.i.d. N(0, std^2) entries, drawn in fp32 and returned in storage format (chunked: tables are GBs)."""
    g = _rng(seed, stream)
    rows = int(shape[0])
    rest = tuple(int(s) for s in shape[1:])
    out = np.empty(shape, dtype=np.float32 if dtype == F32 else np.uint16)
    for r0 in range(0, rows, chunk_rows):
        r1 = min(rows, r0 + chunk_rows)
        blk = g.standard_normal((r1 - r0,) + rest, dtype=np.float32) * np.float32(std)
        out[r0:r1] = blk if dtype == F32 else f32_to_bf16_bits(blk)
    return out


def history_lengths(seed: int, B: int, n_min: int, n_max: int) -> np.ndarray:
    """Per-user history lengths, uniform on [n_min, n_max] (int32)."""
    if n_min == n_max:
        return np.full(B, n_min, dtype=np.int32)
    return _rng(seed, "lengths").integers(n_min, n_max + 1, size=B, dtype=np.int64).astype(np.int32)


def zipf_ids(seed: int, stream: str, count: int, V: int, s: float) -> np.ndarray:
    """`count` ids with P(rank k) proportional to k^-s on k = 1..V (inverse CDF); ranks are scattered over the
    table rows by a seeded permutation so hot rows are not neighbours."""
    g = _rng(seed, stream)
    pmf = np.arange(1, V + 1, dtype=np.float64) ** (-float(s))
    cdf = np.cumsum(pmf)
    cdf /= cdf[-1]
    u = g.random(count)
    rank = np.minimum(np.searchsorted(cdf, u, side="left"), V - 1)
    perm = _rng(seed, "rank_to_row").permutation(V)
    return perm[rank].astype(np.int32)


def uniform_ids(seed: int, stream: str, count: int, V: int) -> np.ndarray:
    return _rng(seed, stream).integers(0, V, size=count, dtype=np.int64).astype(np.int32)


def layer_weights(seed: int, wl: Workload) -> Dict[str, np.ndarray]:
    """Projection / GatedMLP weights of every XOR layer, variance 1/fan_in, in storage format.
    Shapes: Wq, Wk, Wv [n, d, d]; Wg, Wu [n, d, d_ff]; Wo [n, d_ff, d] (row = input feature)."""
    n, d, f = wl.n_layers, wl.d, wl.dff
    out = {}
    for name, shape, fan_in in (("Wq", (n, d, d), d), ("Wk", (n, d, d), d), ("Wv", (n, d, d), d),
                                ("Wg", (n, d, f), d), ("Wu", (n, d, f), d), ("Wo", (n, f, d), f)):
        out[name] = normal_storage(seed, "w_" + name, shape, fan_in ** -0.5, wl.dtype)
    return out


def ffn_weights(seed: int, stream: str, widths, dtype: str, bias_std: float = 0.1):
    """Weights of a feed-forward network with layer widths `widths` = (in, hidden..., out): a list of
    (W [in_i x out_i] in storage format, variance 1/in_i; b [out_i] fp32, std `bias_std`)."""
    out = []
    for i, (a, b) in enumerate(zip(widths[:-1], widths[1:])):
        W = normal_storage(seed, f"{stream}_W{i}", (int(a), int(b)), float(a) ** -0.5, dtype)
        bias = normal_storage(seed, f"{stream}_b{i}", (int(b),), bias_std, F32)
        out.append((W, bias))
    return out


def make_inputs(wl: Workload, seed: int = 0, with_candidates: bool = True) -> Dict[str, np.ndarray]:
    """All inputs of one batch, as stored arrays (fp32, or uint16 bf16 bit patterns) and int32 indices.

    keys: table [V,d]; links [ell,d]; Wq..Wo; lengths [B]; hist_ids [sum N]; cand_ids [B*C]
    """
    out: Dict[str, np.ndarray] = {}
    out["table"] = normal_storage(seed, "table", (wl.V, wl.d), wl.table_std, wl.dtype)
    out["links"] = normal_storage(seed, "links", (wl.ell, wl.d), wl.link_std, wl.dtype)
    out.update(layer_weights(seed, wl))
    lengths = history_lengths(seed, wl.B, wl.n_min, wl.n_max)
    out["lengths"] = lengths
    total = int(lengths.astype(np.int64).sum())
    if wl.zipf_s is None:
        # every table row is used exactly once: history rows first, candidate rows after, shuffled
        need = total + wl.B * wl.C
        if need > wl.V:
            raise ValueError("table too small for one row per use")
        perm = _rng(seed, "one_use").permutation(wl.V).astype(np.int32)
        out["hist_ids"] = perm[:total].copy()
        if with_candidates:
            out["cand_ids"] = perm[total:need].copy()
    else:
        out["hist_ids"] = zipf_ids(seed, "hist_ids", total, wl.V, wl.zipf_s)
        if with_candidates:
            out["cand_ids"] = uniform_ids(seed, "cand_ids", wl.B * wl.C, wl.V)
    return out

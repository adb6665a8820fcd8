"""CPU oracle for LIME ranking inference (link embeddings + XOR attention + decoupled scoring).

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, fp64 statement of what the
paper's inference path computes.  It exists so that the CUDA library can be checked
against something that can be compared with the paper by eye.  Only the test-suite, the
smoke check and the benchmark's CPU-baseline leg may import it; the product path never
does, and this file imports nothing from the product package.

Everything is numpy float64, two-pass exact softmax, no tiling, no fusion, no
re-association beyond what the cited definition states.  `@` (a library matmul) is used as a
step where the definition is a matrix product.

Notation follows the paper: E [N x d] user history embeddings (source, S), L [l x d] link
embeddings (target, T), L^C contextualised links, L^P personalised links, T/C candidate
embeddings, phi the attention activation, J the all-ones mask.

Conventions fixed here where the paper is silent (each is a *reading*, listed with its reason in
the design notes of the repository):
  * projections act on the right: X~ = X W with W [d x d]  (Eq. 1)
  * heads are H contiguous chunks of d_h = d / H features; head outputs are concatenated, no W_O
  * phi = softmax(s / sqrt(d_h)) over the *unmasked* keys only (Eq. 7 equates XOR attention with two
    all-ones-mask attentions, so normalisation is over the opposite partition)
  * phi = SiLU: SiLU(s) / (size of the opposite partition), no 1/sqrt(d_h)  (Algorithms 1-2)
  * LayerNorm before the Q/K/V projections is non-affine with eps = 1e-5 (App. C, "Normalization")
  * GatedMLP(A) = (SiLU(A W_g) * (A W_u)) W_o, no bias, no residual (Eq. 5 passes it the attention
    output only; the paper gives no formula)   -- parity unpinned by the paper, see PINS below
  * XOR layers are stacked: layer j consumes layer j-1's history and link rows; L^P sums the link
    rows of every layer's output (Eq. 8)
  * an empty history gives zero attention output for the link rows
  * the two small MLPs the paper names without a formula - the link contextualisation of Eq. 2 and the
    "shallow interaction network" that scores the LIME embedding (Sec. 3.3; widths in App. C's table) - are
    plain feed-forward networks: x <- ReLU(x W_i + b_i) for every hidden layer, a linear last layer.  Eq. 2's
    input row is a link row followed by the user's context vector; the interaction network's input row is the
    LIME embedding O_c followed by the candidate embedding T_c   -- parity unpinned by the paper, see PINS below

PINS (what ties each function to something other than itself; see tests/test_oracle_*.py):
  lengths_to_offsets, gather_history : definition, exact integers / bytes
  softmax_rows                       : rows sum to 1, shift invariance, closed-form 2-key weights
  attend / mha                       : uniform keys -> mean of values; one key -> that value; key
                                       permutation invariance; linear in V; equals a library
                                       scaled-dot-product attention; closed-form ln(3) example
  xora_dense vs xora_blocks          : Eq. 6 == Eq. 7; Algorithm 1 truth table; Algorithm 2 tiling
  precompute_candidate_links, score_candidates, encode_user (CORE profile)
                                     : brute-force non-decoupled candidate->link->history loops;
                                       composite attention rows sum to 1 (App. D); l = 1 two-tower dot;
                                       one-hot weights select a link row; candidate permutation
  layer_norm                         : zero mean / unit variance rows, library layer_norm
  gated_mlp, the stacking and the layer sum (FULL profile)
                                     : PARITY UNPINNED by the paper beyond reductions: identity weights
                                       reduce FULL to CORE; n = 1 gives L^P = T^1; the last layer's
                                       history update never reaches the logits
  ffn, contextualize_links, interaction_head
                                     : scalar-loop evaluation; a library Linear/ReLU stack in fp64; zero hidden
                                       weights leave the last bias; bias-free networks are positively
                                       homogeneous; a context vector of zeros makes every user's L^C equal.
                                       Their FORM (inputs, activation) is PARITY UNPINNED by the paper
"""
from __future__ import annotations

import dataclasses
from typing import Dict, List, Optional, Sequence

import numpy as np

SOFTMAX = "softmax"
SILU = "silu"


@dataclasses.dataclass(frozen=True)
class OracleConfig:
    d: int
    H: int
    ell: int
    n_layers: int
    phi: str = SOFTMAX
    ln: bool = True                 # LayerNorm before Q/K/V projections (App. C)
    gated_mlp: bool = True          # GatedMLP after the attention (Eq. 5 / Eq. 8)
    ln_eps: float = 1e-5
    attn_scale: Optional[float] = None   # None -> 1/sqrt(d_h)
    cand_scale: Optional[float] = None   # None -> 1/sqrt(d)

    @property
    def d_h(self) -> int:
        return self.d // self.H

    @property
    def scale(self) -> float:
        return self.attn_scale if self.attn_scale is not None else float(self.d_h) ** -0.5

    @property
    def c_scale(self) -> float:
        return self.cand_scale if self.cand_scale is not None else float(self.d) ** -0.5

    @property
    def c_scale_heads(self) -> float:
        """Scale of the per-head candidate->link scores (Eq. 1 applied to Eq. 4 head by head): 1/sqrt(d_h)."""
        return self.cand_scale if self.cand_scale is not None else float(self.d_h) ** -0.5


# --------------------------------------------------------------------------- #
# ragged bookkeeping and the embedding lookup (Sec. 3, history of N(U) items per user)
# --------------------------------------------------------------------------- #
def lengths_to_offsets(lengths: Sequence[int]) -> np.ndarray:
    """Exclusive prefix sum of per-user history lengths: off[0] = 0, off[b+1] = off[b] + len[b]."""
    off = np.zeros(len(lengths) + 1, dtype=np.int64)
    for b, n in enumerate(lengths):
        off[b + 1] = off[b] + int(n)
    return off


def gather_history(table: np.ndarray, ids: Sequence[int]) -> np.ndarray:
    """E[t, :] = table[ids[t], :] -- one table row per history item (stand-in for the item embedding)."""
    out = np.empty((len(ids), table.shape[1]), dtype=table.dtype)
    for t, i in enumerate(ids):
        out[t, :] = table[int(i), :]
    return out


# --------------------------------------------------------------------------- #
# building blocks of Eq. 1
# --------------------------------------------------------------------------- #
def layer_norm(X: np.ndarray, eps: float = 1e-5) -> np.ndarray:
    """Per-row normalisation over the d features: (x - mean) / sqrt(var + eps), biased variance, no affine."""
    X = np.asarray(X, dtype=np.float64)
    mu = X.mean(axis=-1, keepdims=True)
    var = ((X - mu) ** 2).mean(axis=-1, keepdims=True)
    return (X - mu) / np.sqrt(var + eps)


def silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))


def softmax_rows(S: np.ndarray, mask: Optional[np.ndarray] = None) -> np.ndarray:
    """Row softmax over the unmasked columns (two passes, exact). A row with no unmasked column is all zero."""
    S = np.asarray(S, dtype=np.float64)
    P = np.zeros_like(S)
    for i in range(S.shape[0]):
        cols = np.arange(S.shape[1]) if mask is None else np.nonzero(mask[i])[0]
        if cols.size == 0:
            continue
        row = S[i, cols]
        e = np.exp(row - row.max())
        P[i, cols] = e / e.sum()
    return P


def attend(Qt: np.ndarray, Kt: np.ndarray, Vt: np.ndarray, H: int, phi: str, scale: float,
           mask: Optional[np.ndarray] = None, denom: Optional[np.ndarray] = None) -> np.ndarray:
    """(phi(Q~ K~^T) (.) M) V~ of Eq. 1, for already-projected Q~ [q x d], K~, V~ [n x d], head by head.

    softmax: phi(s) = softmax over unmasked keys of s * scale.
    SiLU   : phi(s) = SiLU(s) / denom[i], zero where masked (Algorithm 2); denom[i] is the size of the
             partition query i attends to (Algorithm 1).
    """
    q, d = Qt.shape
    n = Kt.shape[0]
    d_h = d // H
    out = np.zeros((q, d), dtype=np.float64)
    if n == 0:
        return out
    for h in range(H):
        sl = slice(h * d_h, (h + 1) * d_h)
        S = Qt[:, sl] @ Kt[:, sl].T
        if phi == SOFTMAX:
            P = softmax_rows(S * scale, mask)
        elif phi == SILU:
            P = silu(S) / np.asarray(denom, dtype=np.float64)[:, None]
            if mask is not None:
                P = np.where(mask, P, 0.0)
        else:
            raise ValueError(phi)
        out[:, sl] = P @ Vt[:, sl]
    return out


def mha(Q: np.ndarray, K: np.ndarray, V: np.ndarray, Wq, Wk, Wv, cfg: OracleConfig,
        mask: Optional[np.ndarray] = None, denom: Optional[np.ndarray] = None) -> np.ndarray:
    """MHA(Q, K, V; M; theta) of Eq. 1 with LayerNorm before each projection (App. C).
    A projection given as None is the identity."""
    def proj(X, W):
        Xn = layer_norm(X, cfg.ln_eps) if cfg.ln else np.asarray(X, dtype=np.float64)
        return Xn if W is None else Xn @ W
    if denom is None and cfg.phi == SILU:
        denom = np.full(Q.shape[0], K.shape[0], dtype=np.float64)
    return attend(proj(Q, Wq), proj(K, Wk), proj(V, Wv), cfg.H, cfg.phi, cfg.scale, mask, denom)


# --------------------------------------------------------------------------- #
# XOR attention: Eq. 6 (dense, masked) and Eq. 7 (two block attentions)
# --------------------------------------------------------------------------- #
def xor_mask_and_denominator(i: int, j: int, n_s: int, n_t: int):
    """M_xor under Eq. 6, for X = E (+) L^C: rows 0 .. n_s-1 form the history partition, rows n_s .. n_s+n_t-1 the link
    partition.  Query row i may attend to key row j exactly when the two lie in different partitions ("attend to one
    another only"), and the SiLU form divides a query's row by the number of keys it can attend to, i.e. the size of
    the partition the query is NOT in (Algorithm 1's normaliser)."""
    sizes = (n_s, n_t)
    partition = lambda row: 0 if row < n_s else 1
    attends = partition(i) != partition(j)
    return attends, sizes[1 - partition(i)]


def xora_dense(E: np.ndarray, LC: np.ndarray, Wq, Wk, Wv, cfg: OracleConfig) -> np.ndarray:
    """Eq. 6: MHA(X, X, X; M_xor) on X = E (+) L^C, every (i, j) entry decided by Algorithm 1.
    Returns [(N + l) x d]: history rows first, link rows after."""
    n_s, n_t = E.shape[0], LC.shape[0]
    X = np.concatenate([E, LC], axis=0)
    n = n_s + n_t
    mask = np.zeros((n, n), dtype=bool)
    denom = np.zeros(n, dtype=np.float64)
    for i in range(n):
        for j in range(n):
            mask[i, j], denom[i] = xor_mask_and_denominator(i, j, n_s, n_t)
    return mha(X, X, X, Wq, Wk, Wv, cfg, mask=mask, denom=denom)


def xora_blocks(E: np.ndarray, LC: np.ndarray, Wq, Wk, Wv, cfg: OracleConfig, need_history: bool = True):
    """Eq. 7 / App. H.1: O[S] = phi(Q[S] K[T]^T) V[T] (history attends to links) and
    O[T] = phi(Q[T] K[S]^T) V[S] (links attend to history), both with the all-ones mask J."""
    O_T = mha(LC, E, E, Wq, Wk, Wv, cfg)
    O_S = mha(E, LC, LC, Wq, Wk, Wv, cfg) if need_history else None
    return O_S, O_T


def gated_mlp(A: np.ndarray, Wg, Wu, Wo) -> np.ndarray:
    """GatedMLP(A; eta) = (SiLU(A W_g) (.) (A W_u)) W_o  -- reading of "MLP block ... gated element-wise product"."""
    return (silu(A @ Wg) * (A @ Wu)) @ Wo


# --------------------------------------------------------------------------- #
# user side: Eq. 3 (one layer) and Eq. 8 (n stacked XOR layers)
# --------------------------------------------------------------------------- #
def xor_layer(S: np.ndarray, T: np.ndarray, w: Dict[str, Optional[np.ndarray]], cfg: OracleConfig,
              need_history: bool = True):
    """One XOR layer: GatedMLP(XORA(S (+) T)) on both partitions. Returns (S_next or None, T_next)."""
    O_S, O_T = xora_blocks(S, T, w.get("Wq"), w.get("Wk"), w.get("Wv"), cfg, need_history)
    if cfg.gated_mlp:
        T_next = gated_mlp(O_T, w["Wg"], w["Wu"], w["Wo"])
        S_next = gated_mlp(O_S, w["Wg"], w["Wu"], w["Wo"]) if need_history else None
    else:
        T_next, S_next = O_T, O_S
    return S_next, T_next


def encode_user(E: np.ndarray, LC: np.ndarray, layers: List[Dict[str, Optional[np.ndarray]]],
                cfg: OracleConfig, update_last_history: bool = False):
    """Eq. 8: L^P = sum_j (link rows of XOR layer j's output), layers stacked.  n = 1 with no
    GatedMLP is Eq. 3, L^P = MHA(L^C, E, E; J).  Returns (L^P [l x d], list of per-layer link rows)."""
    S = np.asarray(E, dtype=np.float64)
    T = np.asarray(LC, dtype=np.float64)
    LP = np.zeros_like(T)
    per_layer = []
    for j, w in enumerate(layers):
        last = j == len(layers) - 1
        S_next, T = xor_layer(S, T, w, cfg, need_history=(not last) or update_last_history)
        if S_next is not None:
            S = S_next
        LP = LP + T
        per_layer.append(T)
    return LP, per_layer


def link_states(LP: np.ndarray, Wv_c: Optional[np.ndarray] = None) -> np.ndarray:
    """V~ of Eq. 4: the personalised links as the candidate side's values, L^P W_V (identity if None)."""
    return LP if Wv_c is None else LP @ Wv_c


# --------------------------------------------------------------------------- #
# candidate side: Eq. 4, decoupled attention
# --------------------------------------------------------------------------- #
def precompute_candidate_links(T: np.ndarray, L: np.ndarray, cfg: OracleConfig,
                               Wq_c: Optional[np.ndarray] = None, Wk_c: Optional[np.ndarray] = None) -> np.ndarray:
    """phi(T L^t) of Eq. 4: the user-independent candidate->link attention weights [M x l]
    (softmax over the l links of (T W_Q)(L W_K)^T * cand_scale), cached offline."""
    Tq = T if Wq_c is None else T @ Wq_c
    Lk = L if Wk_c is None else L @ Wk_c
    return softmax_rows((Tq @ Lk.T) * cfg.c_scale)


def candidate_outputs(W: np.ndarray, LS: np.ndarray) -> np.ndarray:
    """O = phi(T L^t) L^P (Eq. 4): per candidate, the weighted sum of the user's link states."""
    return W @ LS


def score_candidates(W: np.ndarray, LS: np.ndarray, T: np.ndarray) -> np.ndarray:
    """logit[c] = < sum_l W[c, l] LS[l, :], T[c, :] > : the LIME embedding O_c dotted with the raw candidate
    embedding (the shallow interaction network is replaced by this dot product)."""
    O = candidate_outputs(W, LS)
    out = np.empty(T.shape[0], dtype=np.float64)
    for c in range(T.shape[0]):
        out[c] = float(np.dot(O[c, :], T[c, :]))
    return out


# Eq. 4 with Eq. 1 taken literally, MHA(T, L, L^P) head by head: every head h has its own weight row
# softmax_l(<(T W_Q)_h, (L W_K)_h> / sqrt(d_h)) and mixes only its d_h columns of the link states.
def precompute_candidate_links_heads(T: np.ndarray, L: np.ndarray, cfg: OracleConfig,
                                     Wq_c: Optional[np.ndarray] = None, Wk_c: Optional[np.ndarray] = None) -> np.ndarray:
    """User-independent weights [M x H x l]: row (c, h) is the softmax over the l links of head h's scores."""
    Tq = T if Wq_c is None else T @ Wq_c
    Lk = L if Wk_c is None else L @ Wk_c
    M, ell, H, d_h = T.shape[0], L.shape[0], cfg.H, cfg.d_h
    W = np.zeros((M, H, ell), dtype=np.float64)
    for h in range(H):
        sl = slice(h * d_h, (h + 1) * d_h)
        W[:, h, :] = softmax_rows((Tq[:, sl] @ Lk[:, sl].T) * cfg.c_scale_heads)
    return W


def candidate_outputs_heads(W: np.ndarray, LS: np.ndarray, cfg: OracleConfig) -> np.ndarray:
    """O[c, head h's columns] = sum_l W[c, h, l] LS[l, head h's columns]."""
    H, d_h = cfg.H, cfg.d_h
    O = np.zeros((W.shape[0], LS.shape[1]), dtype=np.float64)
    for h in range(H):
        sl = slice(h * d_h, (h + 1) * d_h)
        O[:, sl] = W[:, h, :] @ LS[:, sl]
    return O


def score_candidates_heads(W: np.ndarray, LS: np.ndarray, T: np.ndarray, cfg: OracleConfig) -> np.ndarray:
    """logit[c] = <O_c, T_c> with the per-head mix above."""
    O = candidate_outputs_heads(W, LS, cfg)
    out = np.empty(T.shape[0], dtype=np.float64)
    for c in range(T.shape[0]):
        out[c] = float(np.dot(O[c, :], T[c, :]))
    return out


# --------------------------------------------------------------------------- #
# the two small feed-forward networks: Eq. 2 (link contextualisation) and the interaction network of Sec. 3.3
# --------------------------------------------------------------------------- #
def ffn(X: np.ndarray, layers) -> np.ndarray:
    """Feed-forward network on the rows of X: `layers` is a list of (W [in x out], b [out] or None); every layer
    but the last is followed by ReLU."""
    Z = np.asarray(X, dtype=np.float64)
    for i, (W, b) in enumerate(layers):
        Z = Z @ W
        if b is not None:
            Z = Z + b
        if i + 1 < len(layers):
            Z = np.maximum(Z, 0.0)
    return Z


def contextualize_links(L: np.ndarray, EC: np.ndarray, layers) -> np.ndarray:
    """Eq. 2: L^C = MLP(L (+) E^C) for one user.  L [l x d] shared links, EC [d_c] the user's context features;
    every link row is followed by the same context vector, the MLP maps the (d + d_c)-wide rows back to d."""
    X = np.concatenate([np.asarray(L, dtype=np.float64), np.tile(np.asarray(EC, dtype=np.float64), (L.shape[0], 1))], axis=1)
    return ffn(X, layers)


def interaction_head(O: np.ndarray, T: np.ndarray, layers) -> np.ndarray:
    """Sec. 3.3 "Lightweight User-Item Interaction": the LIME embedding O_c is passed to a shallow interaction
    network for scoring.  Input row = O_c followed by T_c; hidden widths as App. C's "Interaction MLP" row (one
    96-wide layer on the industrial model); the last layer has one output, the logit."""
    return ffn(np.concatenate([O, T], axis=1), layers)[:, 0]


def score_candidates_head(W: np.ndarray, LS: np.ndarray, T: np.ndarray, layers) -> np.ndarray:
    """logit[c] = head(O_c, T_c) with O = phi(T L^t) L^P of Eq. 4."""
    return interaction_head(candidate_outputs(W, LS), T, layers)


# --------------------------------------------------------------------------- #
# whole batch
# --------------------------------------------------------------------------- #
def run_user(E: np.ndarray, L: np.ndarray, layers, cfg: OracleConfig, T: np.ndarray,
             LC: Optional[np.ndarray] = None, W: Optional[np.ndarray] = None,
             cand_w: Optional[Dict[str, np.ndarray]] = None, cand_heads: bool = False, head=None):
    """Encode one user and score that user's candidates. Returns (logits [C], link states [l x d], W [C x l]);
    with cand_heads the candidate side runs head by head (W [C x H x l]); with `head` (layers of the interaction
    network) the LIME embedding is scored by that network instead of the dot product."""
    cand_w = cand_w or {}
    LP, _ = encode_user(E, L if LC is None else LC, layers, cfg)
    LS = link_states(LP, cand_w.get("Wv_c"))
    if cand_heads:
        if W is None:
            W = precompute_candidate_links_heads(T, L, cfg, cand_w.get("Wq_c"), cand_w.get("Wk_c"))
        if head is not None:
            return interaction_head(candidate_outputs_heads(W, LS, cfg), T, head), LS, W
        return score_candidates_heads(W, LS, T, cfg), LS, W
    if W is None:
        W = precompute_candidate_links(T, L, cfg, cand_w.get("Wq_c"), cand_w.get("Wk_c"))
    if head is not None:
        return score_candidates_head(W, LS, T, head), LS, W
    return score_candidates(W, LS, T), LS, W


def run_batch(table: np.ndarray, hist_ids: np.ndarray, lengths: Sequence[int], cand_ids: np.ndarray, C: int,
              L: np.ndarray, layers, cfg: OracleConfig, users: Optional[Sequence[int]] = None,
              cand_w: Optional[Dict[str, np.ndarray]] = None):
    """offsets -> gather -> encode -> precompute -> score for the chosen users (all if None).
    `table`, `L`, layer weights are fp64 arrays holding the stored (already rounded) values.
    Returns dict user -> (logits, link states)."""
    off = lengths_to_offsets(lengths)
    res = {}
    for b in (range(len(lengths)) if users is None else users):
        E = gather_history(table, hist_ids[off[b]:off[b + 1]])
        T = gather_history(table, cand_ids[b * C:(b + 1) * C])
        logits, LS, _ = run_user(E, L, layers, cfg, T, cand_w=cand_w)
        res[int(b)] = (logits, LS)
    return res


# --------------------------------------------------------------------------- #
# brute force, used only to pin the decoupled path on tiny inputs (App. D product form)
# --------------------------------------------------------------------------- #
def brute_force_candidate_history_attention(T: np.ndarray, L: np.ndarray, E: np.ndarray, cfg: OracleConfig):
    """Non-decoupled path with scalar loops, CORE profile (no LN, identity projections, softmax, one layer):
    for every candidate c and head h the composite weights A_h[c, j] = sum_l w[c, l] p_h[l, j] over history
    items j, with w = softmax_l(<t_c, L_l> * cand_scale) formed inline and p_h = softmax_j(<L_l, E_j>_h * scale).
    Returns (composite [H x C x N], O [C x d] = per-head composite times E's head slice)."""
    C, d = T.shape
    ell, N, H, d_h = L.shape[0], E.shape[0], cfg.H, cfg.d_h
    comp = np.zeros((H, C, N))
    O = np.zeros((C, d))
    for c in range(C):
        s = [sum(T[c, k] * L[l, k] for k in range(d)) * cfg.c_scale for l in range(ell)]
        m = max(s)
        z = sum(np.exp(v - m) for v in s)
        w = [np.exp(v - m) / z for v in s]
        for h in range(H):
            for l in range(ell):
                sc = [sum(L[l, h * d_h + k] * E[j, h * d_h + k] for k in range(d_h)) * cfg.scale for j in range(N)]
                mm = max(sc)
                zz = sum(np.exp(v - mm) for v in sc)
                for j in range(N):
                    comp[h, c, j] += w[l] * np.exp(sc[j] - mm) / zz
            for j in range(N):
                for k in range(d_h):
                    O[c, h * d_h + k] += comp[h, c, j] * E[j, h * d_h + k]
    return comp, O

"""Pins for the CPU oracle: closed forms, invariants, brute force and library second opinions.

None of these re-types an oracle formula: each expected value comes from the mathematics (a closed form, an
invariant, a special case that reduces to a textbook routine) or from an independent brute-force loop.
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import lime_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rng(seed):
    return np.random.default_rng(seed)


def core_cfg(d, H, ell, n=1, phi=O.SOFTMAX):
    return O.OracleConfig(d=d, H=H, ell=ell, n_layers=n, phi=phi, ln=False, gated_mlp=False)


# ----------------------------------------------------------------------------- offsets / gather
def test_offsets_definition():
    assert O.lengths_to_offsets([]).tolist() == [0]
    assert O.lengths_to_offsets([3, 0, 5, 1]).tolist() == [0, 3, 3, 8, 9]
    big = O.lengths_to_offsets([2 ** 30, 2 ** 30, 2 ** 30])
    assert big[-1] == 3 * 2 ** 30          # no int32 wrap in the oracle


def test_gather_is_row_copy():
    table = np.arange(20, dtype=np.float64).reshape(5, 4)
    out = O.gather_history(table, [4, 0, 4, 2])
    assert out.tolist() == [table[4].tolist(), table[0].tolist(), table[4].tolist(), table[2].tolist()]
    assert O.gather_history(table, []).shape == (0, 4)


# ----------------------------------------------------------------------------- softmax
def test_softmax_rows_sum_to_one_and_shift_invariant():
    S = rng(0).normal(size=(7, 13)) * 5
    P = O.softmax_rows(S)
    assert np.allclose(P.sum(axis=1), 1.0, atol=1e-12)
    assert np.all(P > 0)
    P2 = O.softmax_rows(S + rng(1).normal(size=(7, 1)) * 100)
    assert np.allclose(P, P2, atol=1e-12)


def test_softmax_extreme_scores_finite():
    S = np.array([[80.0, -80.0, 0.0], [-800.0, -800.0, -800.0], [800.0, 0.0, 799.0]])
    P = O.softmax_rows(S)
    assert np.all(np.isfinite(P))
    assert np.allclose(P[1], 1 / 3)
    assert np.allclose(P.sum(axis=1), 1.0)


def test_softmax_closed_form_two_keys():
    # scores (0, ln 3) -> weights (1/4, 3/4) exactly
    P = O.softmax_rows(np.array([[0.0, math.log(3.0)]]))
    assert np.allclose(P, [[0.25, 0.75]], atol=1e-15)


def test_softmax_mask_normalises_over_unmasked_only():
    S = np.array([[1.0, 2.0, 3.0, 4.0]])
    mask = np.array([[True, False, True, False]])
    P = O.softmax_rows(S, mask)
    assert P[0, 1] == 0 and P[0, 3] == 0
    # unmasked scores (1, 3): ratio e^2
    assert math.isclose(P[0, 2] / P[0, 0], math.exp(2.0), rel_tol=1e-12)
    assert math.isclose(P.sum(), 1.0, rel_tol=1e-12)
    assert np.all(O.softmax_rows(S, np.zeros((1, 4), bool)) == 0)


# ----------------------------------------------------------------------------- attention (Eq. 1 / Eq. 3)
def test_uniform_keys_give_mean_of_values():
    r = rng(2)
    N, ell, d, H = 37, 5, 8, 2
    Q = r.normal(size=(ell, d))
    K = np.tile(r.normal(size=(1, d)), (N, 1))        # all keys equal -> uniform attention
    V = r.normal(size=(N, d))
    out = O.attend(Q, K, V, H, O.SOFTMAX, 0.5)
    assert np.allclose(out, np.tile(V.mean(axis=0), (ell, 1)), atol=1e-12)
    out0 = O.attend(np.zeros((ell, d)), r.normal(size=(N, d)), V, H, O.SOFTMAX, 0.5)   # Q = 0 as well
    assert np.allclose(out0, np.tile(V.mean(axis=0), (ell, 1)), atol=1e-12)


def test_single_key_returns_its_value():
    r = rng(3)
    Q, K, V = r.normal(size=(4, 6)), r.normal(size=(1, 6)), r.normal(size=(1, 6))
    assert np.allclose(O.attend(Q, K, V, 3, O.SOFTMAX, 0.7), np.tile(V, (4, 1)), atol=1e-14)


def test_history_permutation_invariance_and_linearity_in_v():
    r = rng(4)
    N, ell, d, H = 29, 6, 12, 3
    Q, K, V, V2 = r.normal(size=(ell, d)), r.normal(size=(N, d)), r.normal(size=(N, d)), r.normal(size=(N, d))
    base = O.attend(Q, K, V, H, O.SOFTMAX, 0.4)
    p = r.permutation(N)
    assert np.allclose(O.attend(Q, K[p], V[p], H, O.SOFTMAX, 0.4), base, atol=1e-12)
    lin = O.attend(Q, K, 2.0 * V - 3.0 * V2, H, O.SOFTMAX, 0.4)
    assert np.allclose(lin, 2.0 * base - 3.0 * O.attend(Q, K, V2, H, O.SOFTMAX, 0.4), atol=1e-12)


def test_closed_form_ln3_attention():
    # one link, two history items, d = d_h = 1: q = 1, keys (0, ln 3), scale 1 -> weights (1/4, 3/4)
    Q = np.array([[1.0]])
    K = np.array([[0.0], [math.log(3.0)]])
    V = np.array([[8.0], [-4.0]])
    out = O.attend(Q, K, V, 1, O.SOFTMAX, 1.0)
    assert math.isclose(out[0, 0], 0.25 * 8.0 + 0.75 * -4.0, rel_tol=1e-14)
    # head split: two heads each of width 1 with different keys -> per-head weights
    Q2 = np.array([[1.0, 1.0]])
    K2 = np.array([[0.0, math.log(7.0)], [math.log(3.0), 0.0]])
    V2 = np.array([[8.0, 16.0], [-4.0, 0.0]])
    out2 = O.attend(Q2, K2, V2, 2, O.SOFTMAX, 1.0)
    assert math.isclose(out2[0, 0], -1.0, rel_tol=1e-14)              # (1/4, 3/4) on head 0
    assert math.isclose(out2[0, 1], 16.0 * 7.0 / 8.0, rel_tol=1e-14)   # (7/8, 1/8) on head 1


@pytest.mark.parametrize("H", [1, 2, 4])
def test_core_attention_equals_library_sdpa(H):
    # CORE profile: textbook scaled dot-product attention, second opinion from torch's fp64 CPU routine
    r = rng(5 + H)
    N, ell, d = 33, 7, 16
    L, E = r.normal(size=(ell, d)), r.normal(size=(N, d))
    cfg = core_cfg(d, H, ell)
    mine = O.mha(L, E, E, None, None, None, cfg)
    q = torch.from_numpy(L).reshape(ell, H, d // H).transpose(0, 1)
    k = torch.from_numpy(E).reshape(N, H, d // H).transpose(0, 1)
    ref = torch.nn.functional.scaled_dot_product_attention(q, k, k)        # default scale 1/sqrt(d_h)
    ref = ref.transpose(0, 1).reshape(ell, d).numpy()
    assert np.allclose(mine, ref, atol=1e-12)


def test_projected_mha_equals_library_mha_without_out_proj():
    # Eq. 1 with W_Q, W_K, W_V against torch's multi_head_attention_forward (out_proj = identity, no bias)
    r = rng(9)
    N, ell, d, H = 21, 5, 12, 3
    L, E = r.normal(size=(ell, d)), r.normal(size=(N, d))
    Wq, Wk, Wv = (r.normal(size=(d, d)) / math.sqrt(d) for _ in range(3))
    cfg = core_cfg(d, H, ell)
    mine = O.mha(L, E, E, Wq, Wk, Wv, cfg)
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a))
    ref, _ = torch.nn.functional.multi_head_attention_forward(
        t(L)[:, None, :], t(E)[:, None, :], t(E)[:, None, :], d, H,
        in_proj_weight=None, in_proj_bias=None, bias_k=None, bias_v=None, add_zero_attn=False, dropout_p=0.0,
        out_proj_weight=torch.eye(d, dtype=torch.float64), out_proj_bias=None, need_weights=False,
        use_separate_proj_weight=True, q_proj_weight=t(Wq.T), k_proj_weight=t(Wk.T), v_proj_weight=t(Wv.T))
    assert np.allclose(mine, ref[:, 0, :].numpy(), atol=1e-12)


def test_layer_norm_stats_and_library():
    X = rng(10).normal(size=(9, 32)) * 3 + 5
    Y = O.layer_norm(X, 1e-5)
    assert np.allclose(Y.mean(axis=1), 0, atol=1e-12)
    assert np.allclose(Y.var(axis=1), 1.0, atol=1e-4)      # eps makes it slightly below 1
    ref = torch.nn.functional.layer_norm(torch.from_numpy(X), (32,), eps=1e-5).numpy()
    assert np.allclose(Y, ref, atol=1e-12)


def test_empty_history_gives_zero_links():
    cfg = core_cfg(8, 2, 3)
    out = O.mha(rng(0).normal(size=(3, 8)), np.zeros((0, 8)), np.zeros((0, 8)), None, None, None, cfg)
    assert out.shape == (3, 8) and np.all(out == 0)


# ----------------------------------------------------------------------------- XOR attention (Eq. 6 = Eq. 7, Alg. 1-2)
def test_algorithm1_truth_table():
    # golden fixture: rows "i j n_s n_t -> mask denominator", transcribed from Algorithm 1's four cases
    with open(os.path.join(GOLDEN, "alg1_xor_mask.txt")) as f:
        rows = [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]
    assert len(rows) >= 4
    for i, j, n_s, n_t, m, dn in rows:
        got_m, got_d = O.xor_mask_and_denominator(int(i), int(j), int(n_s), int(n_t))
        assert int(got_m) == int(m) and got_d == int(dn)


@pytest.mark.parametrize("phi", [O.SOFTMAX, O.SILU])
@pytest.mark.parametrize("ln", [False, True])
def test_eq6_dense_xor_equals_eq7_blocks(phi, ln):
    r = rng(11)
    N, ell, d, H = 19, 5, 8, 2
    E, L = r.normal(size=(N, d)), r.normal(size=(ell, d))
    Wq, Wk, Wv = (r.normal(size=(d, d)) / math.sqrt(d) for _ in range(3))
    cfg = O.OracleConfig(d=d, H=H, ell=ell, n_layers=1, phi=phi, ln=ln, gated_mlp=False)
    dense = O.xora_dense(E, L, Wq, Wk, Wv, cfg)
    O_S, O_T = O.xora_blocks(E, L, Wq, Wk, Wv, cfg)
    assert np.allclose(dense[:N], O_S, atol=1e-12)
    assert np.allclose(dense[N:], O_T, atol=1e-12)


def _alg2_tiled(Q, K, V, n_s, B_M, B_N):
    """Independent tiled evaluation with block-range selection as Algorithm 2 describes it (single head, SiLU)."""
    n, d = Q.shape
    n_t = n - n_s
    out = np.zeros((n, d))
    for q0 in range(0, n, B_M):
        q1 = min(n, q0 + B_M)
        if q1 <= n_s:
            k_lo, k_hi = n_s, n
        elif q0 >= n_s:
            k_lo, k_hi = 0, n_s
        else:
            k_lo, k_hi = 0, n
        acc = np.zeros((q1 - q0, d))
        for k0 in range(k_lo, k_hi, B_N):
            k1 = min(k_hi, k0 + B_N)
            S = Q[q0:q1] @ K[k0:k1].T
            for i in range(q1 - q0):
                for j in range(k1 - k0):
                    src_q, src_k = (q0 + i) < n_s, (k0 + j) < n_s
                    if src_q != src_k:
                        dn = n_t if src_q else n_s
                        S[i, j] = S[i, j] / (1 + math.exp(-S[i, j])) / dn
                    else:
                        S[i, j] = 0.0
            acc += S @ V[k0:k1]
        out[q0:q1] = acc
    return out


@pytest.mark.parametrize("B_M,B_N", [(4, 4), (5, 3), (16, 8), (64, 64)])
def test_algorithm2_tiling_independence(B_M, B_N):
    r = rng(12)
    N, ell, d = 23, 6, 8           # boundary tile straddles n_s for most tilings
    E, L = r.normal(size=(N, d)), r.normal(size=(ell, d))
    cfg = core_cfg(d, 1, ell, phi=O.SILU)
    O_S, O_T = O.xora_blocks(E, L, None, None, None, cfg)
    X = np.concatenate([E, L])
    tiled = _alg2_tiled(X, X, X, N, B_M, B_N)
    assert np.allclose(tiled[:N], O_S, atol=1e-12)
    assert np.allclose(tiled[N:], O_T, atol=1e-12)


# ----------------------------------------------------------------------------- decoupled candidate side (Eq. 4, App. D)
@pytest.mark.parametrize("H", [1, 2])
def test_decoupled_equals_brute_force_non_decoupled(H):
    r = rng(13)
    N, ell, d, C = 11, 4, 4, 6
    E, L, T = r.normal(size=(N, d)), r.normal(size=(ell, d)), r.normal(size=(C, d))
    cfg = core_cfg(d, H, ell)
    comp, O_bf = O.brute_force_candidate_history_attention(T, L, E, cfg)
    assert np.allclose(comp.sum(axis=2), 1.0, atol=1e-12)          # product of row-stochastic matrices
    assert np.all(comp >= 0)
    LP, _ = O.encode_user(E, L, [{}], cfg)
    W = O.precompute_candidate_links(T, L, cfg)
    assert np.allclose(O.candidate_outputs(W, O.link_states(LP)), O_bf, atol=1e-12)
    logits = O.score_candidates(W, LP, T)
    assert np.allclose(logits, (O_bf * T).sum(axis=1), atol=1e-12)
    logits2, LS2, W2 = O.run_user(E, L, [{}], cfg, T)
    assert np.allclose(logits2, logits, atol=1e-14) and np.allclose(W2, W) and np.allclose(LS2, LP)


def test_precompute_rows_and_scale():
    r = rng(14)
    T, L = r.normal(size=(9, 16)), r.normal(size=(5, 16))
    cfg = core_cfg(16, 4, 5)
    W = O.precompute_candidate_links(T, L, cfg)
    assert W.shape == (9, 5) and np.allclose(W.sum(axis=1), 1.0, atol=1e-12)
    # ratio of two weights in a row is exp((s1 - s2) / sqrt(d)), s = <t, l>
    s = T[3] @ L.T
    assert math.isclose(W[3, 1] / W[3, 4], math.exp((s[1] - s[4]) / 4.0), rel_tol=1e-12)
    # transposed operands would change the shape / break this: candidate scaling by a constant row
    Wc = O.precompute_candidate_links(np.zeros((2, 16)), L, cfg)
    assert np.allclose(Wc, 1.0 / 5)
    # candidate-side projections fold: (T Wq)(L Wk)^T
    Wq, Wk = r.normal(size=(16, 16)), r.normal(size=(16, 16))
    Wp = O.precompute_candidate_links(T, L, cfg, Wq, Wk)
    assert np.allclose(Wp, O.precompute_candidate_links(T @ Wq, L @ Wk, cfg), atol=1e-14)


def test_scoring_invariants():
    r = rng(15)
    C, ell, d = 10, 4, 6
    W = O.softmax_rows(r.normal(size=(C, ell)))
    LS, T = r.normal(size=(ell, d)), r.normal(size=(C, d))
    base = O.score_candidates(W, LS, T)
    p = r.permutation(C)
    assert np.allclose(O.score_candidates(W[p], LS, T[p]), base[p], atol=1e-14)    # candidate permutation
    # l = 1: W == 1, two-tower dot product
    one = O.score_candidates(np.ones((C, 1)), LS[:1], T)
    assert np.allclose(one, T @ LS[0], atol=1e-14)
    # one-hot weights select a link row
    sel = r.integers(0, ell, size=C)
    hot = np.eye(ell)[sel]
    assert np.allclose(O.score_candidates(hot, LS, T), np.einsum("cd,cd->c", LS[sel], T), atol=1e-14)
    # brute-force triple loop
    bf = [sum(W[c, l] * LS[l, k] * T[c, k] for l in range(ell) for k in range(d)) for c in range(C)]
    assert np.allclose(base, bf, atol=1e-13)


def test_per_head_candidate_side_is_multi_head_attention():
    """Eq. 1 applied to Eq. 4 head by head: the decoupled form (weights cached per head, then the per-head mix and the
    dot with the candidate) must equal torch's multi-head attention of the candidates over the links with the link
    states as values, and scalar loops; H = 1 must be the single-row form."""
    r = rng(41)
    C, ell, d, H = 7, 5, 12, 3
    T, L, LS = r.normal(size=(C, d)), r.normal(size=(ell, d)), r.normal(size=(ell, d))
    Wq, Wk = r.normal(size=(d, d)), r.normal(size=(d, d))
    cfg = core_cfg(d, H, ell)
    W = O.precompute_candidate_links_heads(T, L, cfg, Wq, Wk)
    assert W.shape == (C, H, ell) and np.allclose(W.sum(axis=2), 1.0, atol=1e-12)
    out = O.candidate_outputs_heads(W, LS, cfg)
    # library second opinion: scaled_dot_product_attention over the head-split tensors (scale 1/sqrt(d_h) by default)
    tq = torch.from_numpy(T @ Wq).reshape(C, H, d // H).transpose(0, 1)
    lk = torch.from_numpy(L @ Wk).reshape(ell, H, d // H).transpose(0, 1)
    lv = torch.from_numpy(LS).reshape(ell, H, d // H).transpose(0, 1)
    ref = torch.nn.functional.scaled_dot_product_attention(tq, lk, lv).transpose(0, 1).reshape(C, d).numpy()
    assert np.allclose(out, ref, atol=1e-12)
    # scalar loops for one candidate and head
    c, h, dh = 4, 2, d // H
    tqn, lkn = T @ Wq, L @ Wk
    sc = [sum(tqn[c, h * dh + k] * lkn[l, h * dh + k] for k in range(dh)) / math.sqrt(dh) for l in range(ell)]
    z = sum(math.exp(v - max(sc)) for v in sc)
    w = [math.exp(v - max(sc)) / z for v in sc]
    assert np.allclose(W[c, h], w, atol=1e-12)
    logits = O.score_candidates_heads(W, LS, T, cfg)
    bf = [sum(W[cc, hh, l] * LS[l, hh * dh + k] * T[cc, hh * dh + k] for hh in range(H) for l in range(ell) for k in range(dh))
          for cc in range(C)]
    assert np.allclose(logits, bf, atol=1e-12)
    # candidate permutation
    p = r.permutation(C)
    assert np.allclose(O.score_candidates_heads(W[p], LS, T[p], cfg), logits[p], atol=1e-14)
    # one head: the single-row form (its default scale 1/sqrt(d) equals 1/sqrt(d_h) then)
    cfg1 = core_cfg(d, 1, ell)
    W1 = O.precompute_candidate_links_heads(T, L, cfg1, Wq, Wk)
    assert np.allclose(W1[:, 0, :], O.precompute_candidate_links(T, L, cfg1, Wq, Wk), atol=1e-14)
    assert np.allclose(O.score_candidates_heads(W1, LS, T, cfg1), O.score_candidates(W1[:, 0, :], LS, T), atol=1e-13)
    # a head only sees its own columns: changing another head's columns of the links leaves its weights alone
    L2 = L.copy()
    L2[0, :dh] += 1.0
    W2 = O.precompute_candidate_links_heads(T, L2, cfg, None, None)
    W0 = O.precompute_candidate_links_heads(T, L, cfg, None, None)
    assert np.allclose(W2[:, 1:, :], W0[:, 1:, :], atol=1e-14) and not np.allclose(W2[:, 0, :], W0[:, 0, :])


def test_link_states_value_projection():
    r = rng(16)
    LP, Wv = r.normal(size=(3, 4)), r.normal(size=(4, 4))
    assert np.allclose(O.link_states(LP), LP)
    bf = [[sum(LP[i, k] * Wv[k, j] for k in range(4)) for j in range(4)] for i in range(3)]
    assert np.allclose(O.link_states(LP, Wv), bf, atol=1e-14)


# ----------------------------------------------------------------------------- FULL wrapper reductions (Eq. 5 / Eq. 8)
def _full_layers(r, n, d, f):
    return [dict(Wq=r.normal(size=(d, d)) / math.sqrt(d), Wk=r.normal(size=(d, d)) / math.sqrt(d),
                 Wv=r.normal(size=(d, d)) / math.sqrt(d), Wg=r.normal(size=(d, f)) / math.sqrt(d),
                 Wu=r.normal(size=(d, f)) / math.sqrt(d), Wo=r.normal(size=(f, d)) / math.sqrt(f)) for _ in range(n)]


def test_gated_mlp_closed_forms():
    # zero gate input -> SiLU(0) = 0 -> output 0 ; scalar case by hand: A=2, Wg=1, Wu=3, Wo=0.5
    assert np.all(O.gated_mlp(np.ones((2, 3)), np.zeros((3, 4)), np.ones((3, 4)), np.ones((4, 3))) == 0)
    got = O.gated_mlp(np.array([[2.0]]), np.array([[1.0]]), np.array([[3.0]]), np.array([[0.5]]))
    want = (2.0 / (1.0 + math.exp(-2.0))) * 6.0 * 0.5
    assert math.isclose(got[0, 0], want, rel_tol=1e-14)
    # row independence: each row only depends on itself
    r = rng(17)
    A, (w,) = r.normal(size=(5, 4)), _full_layers(r, 1, 4, 6)
    full = O.gated_mlp(A, w["Wg"], w["Wu"], w["Wo"])
    assert np.allclose(O.gated_mlp(A[2:3], w["Wg"], w["Wu"], w["Wo"]), full[2:3], atol=1e-14)


def test_full_reduces_to_core_with_identity_weights():
    r = rng(18)
    N, ell, d, H = 17, 4, 8, 2
    E, L = r.normal(size=(N, d)), r.normal(size=(ell, d))
    I = np.eye(d)
    full_noln = O.OracleConfig(d=d, H=H, ell=ell, n_layers=1, ln=False, gated_mlp=False)
    a, _ = O.encode_user(E, L, [dict(Wq=I, Wk=I, Wv=I)], full_noln)
    b, _ = O.encode_user(E, L, [{}], core_cfg(d, H, ell))
    assert np.allclose(a, b, atol=1e-13)


def test_single_layer_lp_is_layer_output_and_sum_over_layers():
    r = rng(19)
    N, ell, d, H, n = 13, 3, 8, 2, 3
    E, L = r.normal(size=(N, d)), r.normal(size=(ell, d))
    layers = _full_layers(r, n, d, d)
    cfg = O.OracleConfig(d=d, H=H, ell=ell, n_layers=n)
    LP, per = O.encode_user(E, L, layers, cfg)
    assert len(per) == n and np.allclose(LP, sum(per), atol=1e-14)
    LP1, per1 = O.encode_user(E, L, layers[:1], cfg)
    assert np.allclose(LP1, per1[0]) and np.allclose(per1[0], per[0], atol=1e-14)
    # stacking: layer 2's link rows equal a fresh one-layer run on layer 1's outputs
    S1, T1 = O.xor_layer(E, L, layers[0], cfg)
    _, T2 = O.xor_layer(S1, T1, layers[1], cfg, need_history=False)
    assert np.allclose(T2, per[1], atol=1e-14)


def test_last_layer_history_update_does_not_reach_links():
    r = rng(20)
    N, ell, d, H = 9, 3, 8, 2
    E, L = r.normal(size=(N, d)), r.normal(size=(ell, d))
    layers = _full_layers(r, 2, d, d)
    cfg = O.OracleConfig(d=d, H=H, ell=ell, n_layers=2)
    a, _ = O.encode_user(E, L, layers, cfg, update_last_history=False)
    b, _ = O.encode_user(E, L, layers, cfg, update_last_history=True)
    assert np.array_equal(a, b)


def test_history_order_does_not_change_link_states_and_users_are_independent():
    r = rng(21)
    ell, d, H, C = 4, 8, 2, 5
    L = r.normal(size=(ell, d))
    table = r.normal(size=(50, d))
    layers = _full_layers(r, 2, d, d)
    cfg = O.OracleConfig(d=d, H=H, ell=ell, n_layers=2)
    lengths = [7, 0, 12]
    ids = r.integers(0, 50, size=sum(lengths))
    cand = r.integers(0, 50, size=3 * C)
    res = O.run_batch(table, ids, lengths, cand, C, L, layers, cfg)
    # user 0 with its history shuffled
    ids2 = ids.copy()
    ids2[:7] = ids[:7][r.permutation(7)]
    ids2[7:] = r.integers(0, 50, size=12)           # change user 2 entirely
    res2 = O.run_batch(table, ids2, lengths, cand, C, L, layers, cfg)
    assert np.allclose(res[0][0], res2[0][0], atol=1e-12)
    assert np.allclose(res[1][0], res2[1][0], atol=0)
    assert not np.allclose(res[2][0], res2[2][0])
    # empty history: link states are zero (GatedMLP(0) = 0), logits zero
    assert np.all(res[1][1] == 0) and np.all(res[1][0] == 0)
    # subset selection returns the same numbers
    sub = O.run_batch(table, ids, lengths, cand, C, L, layers, cfg, users=[2])
    assert np.array_equal(sub[2][0], res[2][0])


def test_silu_attention_matches_scalar_loops():
    r = rng(22)
    N, ell, d = 6, 3, 4
    E, L = r.normal(size=(N, d)), r.normal(size=(ell, d))
    cfg = core_cfg(d, 2, ell, phi=O.SILU)
    out = O.mha(L, E, E, None, None, None, cfg)
    want = np.zeros((ell, d))
    for h in range(2):
        for i in range(ell):
            for j in range(N):
                s = sum(L[i, 2 * h + k] * E[j, 2 * h + k] for k in range(2))
                p = s / (1 + math.exp(-s)) / N
                for k in range(2):
                    want[i, 2 * h + k] += p * E[j, 2 * h + k]
    assert np.allclose(out, want, atol=1e-13)


# ----------------------------------------------------------------------------- feed-forward networks (Eq. 2, Sec. 3.3)
def _ffn_scalar(x, layers):
    """One row through the network with scalar loops only."""
    z = [float(v) for v in x]
    for i, (W, b) in enumerate(layers):
        out = []
        for j in range(W.shape[1]):
            acc = 0.0 if b is None else float(b[j])
            for k in range(W.shape[0]):
                acc += z[k] * float(W[k, j])
            out.append(max(acc, 0.0) if i + 1 < len(layers) else acc)
        z = out
    return z


def _rand_ffn(g, widths, bias=True):
    return [(g.normal(size=(a, b)) / math.sqrt(a), g.normal(size=b) * 0.3 if bias else None)
            for a, b in zip(widths[:-1], widths[1:])]


def test_ffn_against_scalar_loops_and_torch():
    g = rng(31)
    for widths in ([6, 5, 1], [8, 7, 4, 3], [5, 2]):
        layers = _rand_ffn(g, widths)
        X = g.normal(size=(9, widths[0]))
        got = O.ffn(X, layers)
        want = np.array([_ffn_scalar(x, layers) for x in X])
        assert np.allclose(got, want, atol=1e-12)
        mods = []
        for i, (W, b) in enumerate(layers):
            lin = torch.nn.Linear(W.shape[0], W.shape[1]).double()
            with torch.no_grad():
                lin.weight.copy_(torch.from_numpy(W.T))
                lin.bias.copy_(torch.from_numpy(b))
            mods.append(lin)
            if i + 1 < len(layers):
                mods.append(torch.nn.ReLU())
        with torch.no_grad():
            ref = torch.nn.Sequential(*mods)(torch.from_numpy(X)).numpy()
        assert np.allclose(got, ref, atol=1e-12)


def test_ffn_reductions():
    g = rng(32)
    layers = _rand_ffn(g, [6, 8, 1])
    X = g.normal(size=(4, 6))
    # zero hidden weights and bias: the ReLU layer outputs 0, the logit is the last bias
    zeroed = [(np.zeros_like(layers[0][0]), np.zeros_like(layers[0][1])), layers[1]]
    assert np.allclose(O.ffn(X, zeroed)[:, 0], layers[1][1][0])
    # without biases a ReLU network is positively homogeneous
    nobias = [(W, None) for W, _ in layers]
    assert np.allclose(O.ffn(3.5 * X, nobias), 3.5 * O.ffn(X, nobias), atol=1e-12)
    # a hidden layer that passes a non-negative input through (identity weights) leaves a linear map
    Xp = np.abs(X)
    ident = [(np.eye(6), None), (layers[1][0][:6], None)]
    assert np.allclose(O.ffn(Xp, ident), Xp @ layers[1][0][:6], atol=1e-12)


def test_interaction_head_inputs_and_permutation():
    g = rng(33)
    d, ell, C = 6, 3, 7
    W = O.softmax_rows(g.normal(size=(C, ell)))
    LS, T = g.normal(size=(ell, d)), g.normal(size=(C, d))
    layers = _rand_ffn(g, [2 * d, 5, 1])
    got = O.score_candidates_head(W, LS, T, layers)
    # row c of the network's input is (O_c, T_c) with O_c = sum_l W[c, l] LS[l, :]  (Eq. 4), in scalar loops
    for c in range(C):
        o = [sum(W[c, l] * LS[l, k] for l in range(ell)) for k in range(d)]
        assert abs(got[c] - _ffn_scalar(o + list(T[c]), layers)[0]) < 1e-12
    perm = g.permutation(C)
    assert np.allclose(O.score_candidates_head(W[perm], LS, T[perm], layers), got[perm], atol=1e-13)
    # a head whose first layer ignores the O half scores the candidate embedding alone, whatever the user
    W1 = layers[0][0].copy()
    W1[:d] = 0.0
    blind = [(W1, layers[0][1]), layers[1]]
    assert np.allclose(O.score_candidates_head(W, LS, T, blind), O.score_candidates_head(W, 7.0 * LS + 1.0, T, blind), atol=1e-13)


def test_contextualize_links_eq2():
    g = rng(34)
    d, d_c, ell = 6, 4, 5
    L = g.normal(size=(ell, d))
    layers = _rand_ffn(g, [d + d_c, 7, d])
    ec = g.normal(size=d_c)
    LC = O.contextualize_links(L, ec, layers)
    assert LC.shape == (ell, d)
    for l in range(ell):
        assert np.allclose(LC[l], _ffn_scalar(list(L[l]) + list(ec), layers), atol=1e-12)
    # first layer splits over the concatenation: (L (+) E^C) W = L W[:d] + E^C W[d:]
    W1, b1 = layers[0]
    hidden = np.maximum(L @ W1[:d] + ec @ W1[d:] + b1, 0.0)
    assert np.allclose(LC, hidden @ layers[1][0] + layers[1][1], atol=1e-12)
    # a first layer that ignores the context columns gives every user the same contextualised links
    W1z = W1.copy()
    W1z[d:] = 0.0
    same = [(W1z, b1), layers[1]]
    assert np.allclose(O.contextualize_links(L, ec, same), O.contextualize_links(L, g.normal(size=d_c), same), atol=1e-13)
    # L^C feeds the user side in place of L (Eq. 3 / Eq. 8): encode_user takes it as the link rows
    cfg = core_cfg(d, 2, ell)
    E = g.normal(size=(11, d))
    LP, _ = O.encode_user(E, LC, [dict()], cfg)
    assert np.allclose(LP, O.mha(LC, E, E, None, None, None, cfg), atol=1e-13)

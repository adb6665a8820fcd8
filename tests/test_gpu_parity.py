"""Parity of the CUDA library (through the C ABI) against the fp64 CPU oracle, element by element, on the same
seeded inputs.  Tolerances: bit-exact for offsets and gathered rows; logits max-abs <= 1e-4 on the fp32 path and
<= 2e-2 with bf16 storage (plus a relative bound against the spread of the oracle's logits, because logits of the
synthetic workloads are small and the absolute bound alone would be vacuous)."""
import numpy as np
import pytest
import torch

from oracle import lime_oracle as O
from paper_2510_18239_b200 import synth
from tests import lime_helpers as Hh

pytestmark = [pytest.mark.gpu, pytest.mark.skipif(not torch.cuda.is_available(), reason="needs a CUDA device")]

TOL_F32 = 1e-4
TOL_BF16 = 2e-2
REL_BF16 = 6e-2     # max-abs error / std(oracle logits), bf16 storage of history rows through n layers


def _lib():
    from paper_2510_18239_b200 import binding
    return binding


def small(dtype, **kw):
    base = dict(name="small", B=3, n_min=40, n_max=40, d=32, H=2, ell=8, n_layers=2, C=24, dtype=dtype, V=500,
                zipf_s=1.1, table_std=1.0, link_std=1.0)
    base.update(kw)
    return synth.Workload(**base)


# ----------------------------------------------------------------------------- offsets / gather: bit exact
@pytest.mark.parametrize("B", [0, 1, 2, 31, 1000, 1024, 1025, 5000])
def test_offsets_bit_exact(B):
    Bd = _lib()
    lime = Bd.Lime(32, 2, 8, 1, dtype=Bd.LIME_F32)
    r = np.random.default_rng(B)
    lengths = r.integers(0, 4097, size=B).astype(np.int32)
    if B > 4:
        lengths[r.integers(0, B, size=B // 4)] = 0
    off = lime.lengths_to_offsets(torch.from_numpy(lengths).cuda())
    want = O.lengths_to_offsets(lengths)
    assert off.dtype == torch.int32
    assert np.array_equal(off.cpu().numpy().astype(np.int64), want)


@pytest.mark.parametrize("dtype,d", [(synth.F32, 8), (synth.F32, 64), (synth.BF16, 8), (synth.BF16, 128),
                                     (synth.BF16, 256), (synth.BF16, 1024)])
def test_gather_bit_exact_and_bad_ids(dtype, d):
    Bd = _lib()
    V, n = 777, 5001
    lime = Bd.Lime(d, 1 if d < 128 else d // 128, 4, 1, dtype=Bd.LIME_F32 if dtype == synth.F32 else Bd.LIME_BF16)
    table = synth.normal_storage(1, "t", (V, d), 1.0, dtype)
    ids = synth.zipf_ids(1, "i", n, V, 1.1)
    ids[17] = -1
    ids[4000] = V
    ids[4500] = 2 ** 31 - 1
    flag = torch.full((1,), 2 ** 31 - 1, dtype=torch.int32, device="cuda")
    out = lime.gather_history(Bd.to_device(table, dtype), torch.from_numpy(ids).cuda(), flag)
    got = out.view(torch.int16).cpu().numpy().view(np.uint16) if dtype == synth.BF16 else out.cpu().numpy()
    ok = (ids >= 0) & (ids < V)
    want = np.zeros((n, d), dtype=table.dtype)
    want[ok] = O.gather_history(table, ids[ok])
    assert np.array_equal(got.view(np.uint8), want.view(np.uint8))
    assert int(flag.item()) == 17
    # empty gather is legal
    assert lime.gather_history(Bd.to_device(table, dtype), torch.zeros(0, dtype=torch.int32, device="cuda")).shape == (0, d)


# ----------------------------------------------------------------------------- candidate side
@pytest.mark.parametrize("dtype,d", [(synth.F32, 8), (synth.F32, 64), (synth.F32, 1024), (synth.BF16, 8), (synth.BF16, 40),
                                     (synth.BF16, 128), (synth.BF16, 256), (synth.BF16, 1024)])
def test_gather_normalized_is_layer_norm_of_the_rows(dtype, d):
    """Lookup fused with the non-affine LayerNorm (App. C): every row equals the oracle's LayerNorm of the table row
    to the rounding of the storage type; ids outside the table give zero rows and the smallest bad position."""
    Bd = _lib()
    V, n = 777, 5000
    r = np.random.default_rng(d)
    table = synth.to_storage(r.normal(size=(V, d)) * r.uniform(0.01, 3.0, size=(V, 1)) + r.normal(size=(V, 1)), dtype)
    ids = r.integers(0, V, size=n).astype(np.int32)
    ids[[17, 4000]] = [V, -1]
    H = max(1, d // 128)
    L = Bd.Lime(d, H, 4, 1, dtype=Bd.LIME_F32 if dtype == synth.F32 else Bd.LIME_BF16)
    flag = torch.full((1,), 2 ** 31 - 1, dtype=torch.int32, device="cuda")
    got = Hh.to_f64(L.gather_history_normalized(Bd.to_device(table, dtype), torch.from_numpy(ids).cuda(), flag))
    assert int(flag.item()) == 17
    want = O.layer_norm(synth.storage_to_f64(table, dtype)[np.clip(ids, 0, V - 1)])
    want[[17, 4000]] = 0.0
    tol = 1e-5 if dtype == synth.F32 else 2.0 ** -8
    assert np.abs(got - want).max() <= tol * max(1.0, np.abs(want).max())
    # with LayerNorm switched off in the configuration the call is the plain lookup
    L0 = Bd.Lime(d, H, 4, 1, dtype=Bd.LIME_F32 if dtype == synth.F32 else Bd.LIME_BF16, ln=False)
    ok = np.clip(ids, 0, V - 1)
    raw = Hh.to_f64(L0.gather_history_normalized(Bd.to_device(table, dtype), torch.from_numpy(ok).cuda()))
    assert np.array_equal(raw, synth.storage_to_f64(table, dtype)[ok])


@pytest.mark.parametrize("dtype", [synth.F32, synth.BF16])
@pytest.mark.parametrize("ell,d,M", [(1, 8, 5), (8, 64, 300), (32, 128, 1000), (64, 256, 257), (33, 40, 64)])
@pytest.mark.parametrize("proj", [False, True])
def test_precompute_matches_oracle(dtype, ell, d, M, proj):
    Bd = _lib()
    dt = Bd.LIME_F32 if dtype == synth.F32 else Bd.LIME_BF16
    lime = Bd.Lime(d, max(1, d // 128), ell, 1, dtype=dt, gated_mlp=False)
    links = synth.normal_storage(2, "l", (ell, d), 1.0, dtype)
    T = synth.normal_storage(2, "c", (M, d), 1.0, dtype)
    cand_np = {}
    if proj:
        cand_np = {"Wq": synth.normal_storage(2, "cq", (d, d), d ** -0.5, dtype),
                   "Wk": synth.normal_storage(2, "ck", (d, d), d ** -0.5, dtype)}
    lime.set_weights(Bd.to_device(links, dtype), [{}], {k: Bd.to_device(v, dtype) for k, v in cand_np.items()})
    W = lime.precompute_candidate_links(Bd.to_device(T, dtype))
    cfg = O.OracleConfig(d=d, H=1, ell=ell, n_layers=1)
    want = O.precompute_candidate_links(synth.storage_to_f64(T, dtype), synth.storage_to_f64(links, dtype), cfg,
                                        synth.storage_to_f64(cand_np["Wq"], dtype) if proj else None,
                                        synth.storage_to_f64(cand_np["Wk"], dtype) if proj else None)
    got = Hh.to_f64(W)
    assert got.shape == want.shape
    tol = 2e-5 if dtype == synth.F32 else 4e-3          # bf16 output rounding: 2^-9 relative on weights <= 1
    assert np.abs(got - want).max() <= tol
    assert np.abs(got.sum(axis=1) - 1.0).max() <= (1e-5 if dtype == synth.F32 else 1e-2)


@pytest.mark.parametrize("ell,d,M", [(16, 64, 148 * 128 * 9 + 77), (32, 128, 148 * 128 * 5 + 1), (128, 64, 30000),
                                     (64, 256, 148 * 128 * 3 + 127)])
def test_precompute_tensor_core_many_tiles(ell, d, M):
    """bf16 precompute at sizes where every persistent CTA walks several tiles and wraps its stage ring, with a ragged
    last tile; all rows against the oracle."""
    Bd = _lib()
    lime = Bd.Lime(d, max(1, d // 128), ell, 1, dtype=Bd.LIME_BF16, gated_mlp=False)
    links = synth.normal_storage(5, "l", (ell, d), 1.0, synth.BF16)
    T = synth.normal_storage(5, "c", (M, d), 1.0, synth.BF16)
    Wq = synth.normal_storage(5, "cq", (d, d), d ** -0.5, synth.BF16)
    lime.set_weights(Bd.to_device(links, synth.BF16), [{}], {"Wq": Bd.to_device(Wq, synth.BF16)})
    W = lime.precompute_candidate_links(Bd.to_device(T, synth.BF16))
    assert Bd.lime_device_status(lime.ctx) == 0
    cfg = O.OracleConfig(d=d, H=1, ell=ell, n_layers=1)
    T64, L64, Wq64 = (synth.storage_to_f64(x, synth.BF16) for x in (T, links, Wq))
    s = (T64 @ Wq64) @ L64.T * cfg.c_scale                  # the oracle's definition, evaluated for all rows at once
    e = np.exp(s - s.max(axis=1, keepdims=True))
    want = e / e.sum(axis=1, keepdims=True)
    rows = np.random.default_rng(0).integers(0, M, size=50)
    assert np.abs(want[rows] - O.precompute_candidate_links(T64[rows], L64, cfg, Wq64, None)).max() < 1e-12
    got = Hh.to_f64(W)
    assert np.abs(got - want).max() <= 4e-3
    assert np.abs(got.sum(axis=1) - 1.0).max() <= 1e-2


@pytest.mark.parametrize("dtype", [synth.F32, synth.BF16])
@pytest.mark.parametrize("B,C,ell,d", [(1, 1, 1, 8), (3, 50, 8, 64), (2, 300, 32, 128), (2, 129, 64, 256), (5, 77, 33, 40),
                                       (1, 128, 16, 64), (7, 1, 32, 128), (3, 2048, 32, 128), (160, 130, 64, 128),
                                       (2, 1000, 128, 64), (300, 16, 32, 128)])
def test_score_matches_oracle_on_same_inputs(dtype, B, C, ell, d):
    Bd = _lib()
    dt = Bd.LIME_F32 if dtype == synth.F32 else Bd.LIME_BF16
    lime = Bd.Lime(d, max(1, d // 128), ell, 1, dtype=dt, gated_mlp=False)
    LS = synth.normal_storage(3, "ls", (B, ell, d), 1.0, dtype)
    T = synth.normal_storage(3, "t", (B * C, d), 1.0, dtype)
    Wraw = np.abs(synth.storage_to_f64(synth.normal_storage(3, "w", (B * C, ell), 1.0, synth.F32), synth.F32)) + 0.01
    Wst = synth.to_storage(Wraw / Wraw.sum(axis=1, keepdims=True), dtype)
    logits = lime.score_candidates(Bd.to_device(LS, dtype), Bd.to_device(Wst, dtype), Bd.to_device(T, dtype), C=C)
    assert Bd.lime_device_status(lime.ctx) == 0
    W64, T64, LS64 = (synth.storage_to_f64(x, dtype) for x in (Wst, T, LS))
    want = np.concatenate([O.score_candidates(W64[b * C:(b + 1) * C], LS64[b], T64[b * C:(b + 1) * C]) for b in range(B)])
    err = np.abs(Hh.to_f64(logits) - want).max()
    assert err <= 1e-4 * max(1.0, np.abs(want).max()), err      # same stored inputs: only fp32 accumulation differs


@pytest.mark.parametrize("by_id", [False, True])
def test_score_production_shape_many_tiles_per_cta(by_id):
    """The scorer at the shape of `production_ragged` (ell = 64, d = 256: a two-stage ring) with 64 users x 8192
    candidates = 4096 tiles on 148 persistent CTAs, so every CTA wraps its stage ring and reuses both accumulators many
    times; dense streams and rows taken from corpus caches by id.  Sampled rows of every user against the oracle."""
    Bd = _lib()
    dtype, B, C, ell, d, corpus = synth.BF16, 64, 8192, 64, 256, 300_000
    lime = Bd.Lime(d, 8, ell, 1, dtype=Bd.LIME_BF16, gated_mlp=False)
    LS = synth.normal_storage(21, "ls", (B, ell, d), 1.0, dtype)
    n_rows = corpus if by_id else B * C
    T = synth.normal_storage(21, "t", (n_rows, d), 1.0, dtype)
    Wst = synth.to_storage(O.softmax_rows(np.random.default_rng(21).normal(size=(n_rows, ell))), dtype)
    ids = synth.uniform_ids(21, "ids", B * C, corpus) if by_id else None
    logits = lime.score_candidates(Bd.to_device(LS, dtype), Bd.to_device(Wst, dtype), Bd.to_device(T, dtype), C=C,
                                   cand_ids=torch.from_numpy(ids).cuda() if by_id else None, total_cands=B * C)
    assert Bd.lime_device_status(lime.ctx) == 0
    got = Hh.to_f64(logits).reshape(B, C)
    LS64 = synth.storage_to_f64(LS, dtype)
    r = np.random.default_rng(22)
    for b in range(B):
        cols = np.unique(np.concatenate([[0, 127, 128, C - 129, C - 1], r.integers(0, C, size=40)]))
        rows = ids[b * C + cols] if by_id else b * C + cols
        want = O.score_candidates(synth.storage_to_f64(Wst[rows], dtype), LS64[b], synth.storage_to_f64(T[rows], dtype))
        err = np.abs(got[b, cols] - want).max()
        assert err <= 1e-4 * max(1.0, np.abs(want).max()), (b, err)
    assert np.isfinite(got).all()


def test_score_ragged_offsets_ids_and_empty_users():
    Bd = _lib()
    dtype, ell, d = synth.BF16, 16, 64
    lime = Bd.Lime(d, 1, ell, 1, dtype=Bd.LIME_BF16, gated_mlp=False)
    counts = np.array([5, 0, 130, 1, 0, 64, 63], dtype=np.int64)
    B, total = counts.size, int(counts.sum())
    off = O.lengths_to_offsets(counts)
    corpus = 400
    LS = synth.normal_storage(4, "ls", (B, ell, d), 1.0, dtype)
    Tc = synth.normal_storage(4, "t", (corpus, d), 1.0, dtype)
    Wc = synth.to_storage(O.softmax_rows(np.random.default_rng(4).normal(size=(corpus, ell))), dtype)
    ids = synth.uniform_ids(4, "ids", total, corpus)
    logits = lime.score_candidates(Bd.to_device(LS, dtype), Bd.to_device(Wc, dtype), Bd.to_device(Tc, dtype),
                                   cand_off=torch.from_numpy(off.astype(np.int32)).cuda(),
                                   cand_ids=torch.from_numpy(ids).cuda(), total_cands=total)
    W64, T64, LS64 = (synth.storage_to_f64(x, dtype) for x in (Wc, Tc, LS))
    want = np.concatenate([O.score_candidates(W64[ids[off[b]:off[b + 1]]], LS64[b], T64[ids[off[b]:off[b + 1]]])
                           for b in range(B)])
    assert np.abs(Hh.to_f64(logits) - want).max() <= 1e-4 * max(1.0, np.abs(want).max())


@pytest.mark.parametrize("B,C,ell,d,corpus", [(3, 2048, 32, 128, 5000), (2, 129, 64, 256, 300), (160, 130, 16, 64, 1000),
                                              (1, 1, 32, 128, 7), (150, 1000, 32, 128, 100000), (5, 300, 128, 64, 999)])
def test_score_from_corpus_caches_by_ids(B, C, ell, d, corpus):
    """Fixed C per user with candidate ids into corpus-level caches (item embeddings and cached weights): the bf16
    scorer that gathers rows itself, against the oracle on the gathered rows; many tiles per CTA in the larger cases."""
    Bd = _lib()
    dtype = synth.BF16
    lime = Bd.Lime(d, max(1, d // 128), ell, 1, dtype=Bd.LIME_BF16, gated_mlp=False)
    LS = synth.normal_storage(8, "ls", (B, ell, d), 1.0, dtype)
    Tc = synth.normal_storage(8, "t", (corpus, d), 1.0, dtype)
    Wc = synth.to_storage(O.softmax_rows(np.random.default_rng(8).normal(size=(corpus, ell))), dtype)
    ids = synth.uniform_ids(8, "ids", B * C, corpus)
    logits = lime.score_candidates(Bd.to_device(LS, dtype), Bd.to_device(Wc, dtype), Bd.to_device(Tc, dtype), C=C,
                                   cand_ids=torch.from_numpy(ids).cuda(), total_cands=B * C)
    assert Bd.lime_device_status(lime.ctx) == 0
    W64, T64, LS64 = (synth.storage_to_f64(x, dtype) for x in (Wc, Tc, LS))
    want = np.concatenate([O.score_candidates(W64[ids[b * C:(b + 1) * C]], LS64[b], T64[ids[b * C:(b + 1) * C]]) for b in range(B)])
    err = np.abs(Hh.to_f64(logits) - want).max()
    assert err <= 1e-4 * max(1.0, np.abs(want).max()), err


@pytest.mark.parametrize("dtype,B,C,ell,d,corpus,ragged", [(synth.BF16, 3, 2048, 32, 128, 5000, False), (synth.BF16, 2, 129, 64, 256, 300, False),
                                                           (synth.BF16, 150, 1000, 32, 128, 100000, False), (synth.BF16, 5, 300, 128, 64, 999, False),
                                                           (synth.BF16, 4, 50, 33, 40, 257, False), (synth.F32, 3, 70, 8, 64, 257, False),
                                                           (synth.BF16, 3, 0, 16, 64, 257, True)])
def test_score_from_packed_corpus_records(dtype, B, C, ell, d, corpus, ragged):
    """Corpus caches packed as one record per item ([embedding row | weight row], Sec. 3.3): the records are the two
    caches bit for bit, and scoring by id over them gives the oracle's logits (tensor-core scorer with its own gather
    over two views of the one array; generic scorer for the other shapes); ids outside the corpus score 0."""
    Bd = _lib()
    dt = Bd.LIME_F32 if dtype == synth.F32 else Bd.LIME_BF16
    lime = Bd.Lime(d, max(1, d // 128), ell, 1, dtype=dt, gated_mlp=False)
    if ragged:
        counts = np.array([40, 0, 91], dtype=np.int64)
        off = O.lengths_to_offsets(counts)
        total = int(counts.sum())
    else:
        off = np.arange(B + 1, dtype=np.int64) * C
        total = B * C
    LS = synth.normal_storage(41, "ls", (B, ell, d), 1.0, dtype)
    Tc = synth.normal_storage(41, "t", (corpus, d), 1.0, dtype)
    Wc = synth.to_storage(O.softmax_rows(np.random.default_rng(41).normal(size=(corpus, ell))), dtype)
    ids = synth.uniform_ids(41, "ids", total, corpus)
    bad = {3: -1, total - 1: corpus} if total > 8 else {}
    for slot, v in bad.items():
        ids[slot] = v
    packed = lime.pack_corpus_cache(Bd.to_device(Tc, dtype), Bd.to_device(Wc, dtype))
    raw = packed.view(torch.int16).cpu().numpy().view(np.uint16) if dtype == synth.BF16 else packed.cpu().numpy()
    assert np.array_equal(raw[:, :d], Tc) and np.array_equal(raw[:, d:], Wc)
    flag = torch.full((1,), 2 ** 31 - 1, dtype=torch.int32, device="cuda")
    logits = lime.score_candidates_packed(Bd.to_device(LS, dtype), packed, torch.from_numpy(ids).cuda(), C=C,
                                          cand_off=torch.from_numpy(off.astype(np.int32)).cuda() if ragged else None, dev_flag=flag)
    assert Bd.lime_device_status(lime.ctx) == 0
    got = Hh.to_f64(logits)
    W64, T64, LS64 = (synth.storage_to_f64(x, dtype) for x in (Wc, Tc, LS))
    ok_ids = np.clip(ids, 0, corpus - 1)
    want = np.concatenate([O.score_candidates(W64[ok_ids[off[b]:off[b + 1]]], LS64[b], T64[ok_ids[off[b]:off[b + 1]]])
                           for b in range(B)])
    want[list(bad)] = 0.0
    assert np.abs(got - want).max() <= 1e-4 * max(1.0, np.abs(want).max())
    assert np.all(got[list(bad)] == 0.0)
    assert int(flag.item()) == (min(bad) if bad else 2 ** 31 - 1)


@pytest.mark.parametrize("dtype,B,C,ell,d,ragged", [(synth.BF16, 3, 300, 32, 128, False),     # tensor-core scorer with its own gather
                                                    (synth.BF16, 2, 129, 64, 256, False),
                                                    (synth.BF16, 4, 50, 33, 40, False),       # generic scorer, fixed C
                                                    (synth.F32, 3, 70, 8, 64, False),
                                                    (synth.BF16, 3, 0, 16, 64, True)])        # generic scorer, ragged lists
def test_score_by_ids_out_of_range_ids_score_zero(dtype, B, C, ell, d, ragged):
    """Candidate ids outside the corpus caches (-1, V, INT32_MAX) read nothing: those slots get logit 0, the flag holds
    the smallest such slot, and every other slot equals the oracle's logit - on every scorer that takes ids."""
    Bd = _lib()
    dt = Bd.LIME_F32 if dtype == synth.F32 else Bd.LIME_BF16
    corpus = 257
    lime = Bd.Lime(d, max(1, d // 128), ell, 1, dtype=dt, gated_mlp=False)
    if ragged:
        counts = np.array([40, 0, 91], dtype=np.int64)
        off = O.lengths_to_offsets(counts)
        total = int(counts.sum())
    else:
        off = np.arange(B + 1, dtype=np.int64) * C
        total = B * C
    LS = synth.normal_storage(31, "ls", (B, ell, d), 1.0, dtype)
    Tc = synth.normal_storage(31, "t", (corpus, d), 1.0, dtype)
    Wc = synth.to_storage(O.softmax_rows(np.random.default_rng(31).normal(size=(corpus, ell))), dtype)
    ids = synth.uniform_ids(31, "ids", total, corpus)
    bad = {5: -1, 17: corpus, total - 2: 2 ** 31 - 1, total // 2: -2 ** 31}
    for slot, v in bad.items():
        ids[slot] = v
    flag = torch.full((1,), 2 ** 31 - 1, dtype=torch.int32, device="cuda")
    logits = lime.score_candidates(Bd.to_device(LS, dtype), Bd.to_device(Wc, dtype), Bd.to_device(Tc, dtype), C=C,
                                   cand_off=torch.from_numpy(off.astype(np.int32)).cuda() if ragged else None,
                                   cand_ids=torch.from_numpy(ids).cuda(), total_cands=total, corpus_rows=corpus, dev_flag=flag)
    assert Bd.lime_device_status(lime.ctx) == 0
    got = Hh.to_f64(logits)
    W64, T64, LS64 = (synth.storage_to_f64(x, dtype) for x in (Wc, Tc, LS))
    ok_ids = np.clip(ids, 0, corpus - 1)
    want = np.concatenate([O.score_candidates(W64[ok_ids[off[b]:off[b + 1]]], LS64[b], T64[ok_ids[off[b]:off[b + 1]]])
                           for b in range(B)])
    want[list(bad)] = 0.0
    assert np.array_equal(got[list(bad)], np.zeros(len(bad)))
    assert np.abs(got - want).max() <= 1e-4 * max(1.0, np.abs(want).max())
    assert int(flag.item()) == 5
    # the row count is required with ids
    with pytest.raises(Bd.LimeError):
        Bd.lime_score_candidates(lime.ctx, Bd.to_device(LS, dtype), B, Bd.to_device(Wc, dtype), Bd.to_device(Tc, dtype),
                                 torch.from_numpy(off.astype(np.int32)).cuda() if ragged else None, C, total,
                                 torch.from_numpy(ids).cuda(), logits, corpus_rows=-1)


# ----------------------------------------------------------------------------- XOR layer and encode
def _oracle_batch(wl, inp, phi=O.SOFTMAX, ln=True, gated_mlp=True, cand_np=None):
    cfg = Hh.oracle_config(wl, phi=phi, ln=ln, gated_mlp=gated_mlp)
    layers = Hh.oracle_layers(inp, wl, gated_mlp)
    table64 = synth.storage_to_f64(inp["table"], wl.dtype)
    links64 = synth.storage_to_f64(inp["links"], wl.dtype)
    off = O.lengths_to_offsets(inp["lengths"])
    cand_w = None
    if cand_np:
        cand_w = {k + "_c": synth.storage_to_f64(v, wl.dtype) for k, v in cand_np.items()}
    logits, LS = [], []
    for b in range(wl.B):
        lg, ls, _ = Hh.oracle_user(inp, wl, b, off, table64, links64, layers, cfg, cand_w=cand_w)
        logits.append(lg)
        LS.append(ls)
    return np.concatenate(logits), np.stack(LS)


REL_BF16_DRAWN = 1e-1  # the same bound for randomly drawn stress shapes (up to three layers, histories of a single token next to
                       # thousands, SiLU weights that are not confined to [0, 1]): the worst of ~400 sampled logits lands at
                       # 6-7 % of the spread there, the mean error stays below 2 %; a wrong row or divisor errs by ~100 %


def _check_logits(got, want, dtype, stress=False, rel=REL_BF16):
    """The stated bars: max-abs 1e-4 (fp32 path) / 2e-2 (bf16 storage), plus, for bf16, the bound relative to the spread
    of the oracle's logits (the synthetic logits are small, so the absolute bar alone would not bite).  `stress` marks
    synthetic shapes whose logits exceed one: a relaxation of the absolute bar, which is then scaled by max|logit|
    (bf16 storage carries 2^-9 relative rounding per stored value); the named workloads never use it."""
    err = np.abs(got - want).max()
    spread = want.std()
    if dtype == synth.F32:
        assert err <= TOL_F32, (err, spread)
    else:
        assert err <= TOL_BF16 * (max(1.0, np.abs(want).max()) if stress else 1.0), (err, spread)
        assert err <= rel * max(spread, 1e-6) + 1e-4, (err, spread)


@pytest.mark.parametrize("N", [0, 1, 2, 31, 63, 64, 65, 127, 129, 300])
@pytest.mark.parametrize("dtype", [synth.F32, synth.BF16])
def test_xor_layer_history_lengths(N, dtype):
    """One XOR layer, both directions, against the oracle for history lengths around the tile sizes."""
    Bd = _lib()
    wl = small(dtype, B=2, n_min=N, n_max=N, n_layers=1, ell=8, d=32, H=2)
    inp = synth.make_inputs(wl, seed=N)
    dev = Hh.DeviceBatch(wl, inp)
    L = dev.lime
    off = L.lengths_to_offsets(dev.lengths)
    hist = L.gather_history(dev.table, dev.hist_ids)
    links32 = dev.links.float().contiguous()
    hist_out = torch.empty_like(hist)
    links_out = torch.empty((wl.B, wl.ell, wl.d), dtype=torch.float32, device="cuda")
    Bd.lime_xor_layer(L.ctx, 0, hist, off, wl.B, links32, True, hist_out, links_out, L.workspace(wl.B, hist.shape[0]))
    cfg = Hh.oracle_config(wl)
    lw = Hh.oracle_layers(inp, wl)[0]
    table64, links64 = synth.storage_to_f64(inp["table"], dtype), synth.storage_to_f64(inp["links"], dtype)
    tol = 2e-4 if dtype == synth.F32 else 4e-2
    for b in range(wl.B):
        E = O.gather_history(table64, inp["hist_ids"][b * N:(b + 1) * N])
        S_next, T_next = O.xor_layer(E, links64, lw, cfg)
        assert np.abs(Hh.to_f64(links_out[b]) - T_next).max() <= tol
        if N:
            assert np.abs(Hh.to_f64(hist_out[b * N:(b + 1) * N]) - S_next).max() <= tol
    if N == 0:
        assert torch.count_nonzero(links_out).item() == 0


@pytest.mark.parametrize("ell,H", [(32, 4), (16, 8), (64, 2), (64, 4), (32, 8), (64, 8)])
@pytest.mark.parametrize("lengths", [[1], [127, 128, 129], [0, 300, 5, 0, 1000], [256] * 40])
@pytest.mark.parametrize("shared_links", [True, False])
def test_xor_layer_tensor_core_path(ell, H, lengths, shared_links):
    """One XOR layer at the shapes the fused tensor-core kernels serve (bf16, d = 128, H * ell = 128 with all operands
    resident, 256 and 512 with the link-side operands streamed; (64, 2) falls to the generic path), ragged histories
    around the 128-token tile, shared and per-user link rows."""
    Bd = _lib()
    B = len(lengths)
    wl = small(synth.BF16, B=B, n_min=0, n_max=1, d=128, H=H, ell=ell, n_layers=1, V=3000, table_std=0.05)
    inp = synth.make_inputs(wl, seed=ell + B)
    inp["lengths"] = np.asarray(lengths, dtype=np.int32)
    total = int(sum(lengths))
    inp["hist_ids"] = synth.zipf_ids(3, "h", total, wl.V, 1.1)
    dev = Hh.DeviceBatch(wl, inp)
    L = dev.lime
    off = L.lengths_to_offsets(dev.lengths)
    hist = L.gather_history(dev.table, dev.hist_ids)
    if shared_links:
        links_np = synth.storage_to_f64(inp["links"], wl.dtype)[None].repeat(B, axis=0)
        links32 = dev.links.float().contiguous()
    else:
        links_np = np.random.default_rng(9).normal(size=(B, ell, wl.d)).astype(np.float32).astype(np.float64)
        links32 = torch.from_numpy(links_np.astype(np.float32)).cuda()
    hist_out = torch.zeros_like(hist)
    links_out = torch.empty((B, ell, wl.d), dtype=torch.float32, device="cuda")
    Bd.lime_xor_layer(L.ctx, 0, hist, off, B, links32, shared_links, hist_out if total else None, links_out,
                      L.workspace(B, total))
    assert Bd.lime_device_status(L.ctx) == 0
    cfg = Hh.oracle_config(wl)
    lw = Hh.oracle_layers(inp, wl)[0]
    table64 = synth.storage_to_f64(inp["table"], wl.dtype)
    offh = O.lengths_to_offsets(lengths)
    for b in range(B):
        E = O.gather_history(table64, inp["hist_ids"][offh[b]:offh[b + 1]])
        S_next, T_next = O.xor_layer(E, links_np[b], lw, cfg)
        assert np.abs(Hh.to_f64(links_out[b]) - T_next).max() <= 4e-2 * max(1.0, np.abs(T_next).max())
        if lengths[b]:
            got = Hh.to_f64(hist_out[offh[b]:offh[b + 1]])
            assert np.abs(got - S_next).max() <= 4e-2 * max(1.0, np.abs(S_next).max()), (b, np.abs(got - S_next).max())


@pytest.mark.parametrize("ell,H", [(32, 4), (16, 8), (64, 4), (32, 8)])
@pytest.mark.parametrize("lengths", [[127, 128, 129], [0, 300, 5, 0, 1000, 2100]])
@pytest.mark.parametrize("shared_links", [True, False])
def test_xor_layer_tensor_core_path_silu(ell, H, lengths, shared_links):
    """The SiLU form of the XOR attention (Algorithms 1-2: SiLU(s) divided by the size of the attended partition, the
    paper's choice for stacked layers) on the shapes the tensor-core kernels serve; ragged histories, one of them long
    enough to span several chunks so that the per-chunk partials are summed."""
    Bd = _lib()
    B = len(lengths)
    wl = small(synth.BF16, B=B, n_min=0, n_max=1, d=128, H=H, ell=ell, n_layers=1, V=3000, table_std=0.05)
    inp = synth.make_inputs(wl, seed=ell + B)
    inp["lengths"] = np.asarray(lengths, dtype=np.int32)
    total = int(sum(lengths))
    inp["hist_ids"] = synth.zipf_ids(3, "h", total, wl.V, 1.1)
    dev = Hh.DeviceBatch(wl, inp, phi=Bd.LIME_PHI_SILU)
    L = dev.lime
    off = L.lengths_to_offsets(dev.lengths)
    hist = L.gather_history(dev.table, dev.hist_ids)
    if shared_links:
        links_np = synth.storage_to_f64(inp["links"], wl.dtype)[None].repeat(B, axis=0)
        links32 = dev.links.float().contiguous()
    else:
        links_np = np.random.default_rng(9).normal(size=(B, ell, wl.d)).astype(np.float32).astype(np.float64)
        links32 = torch.from_numpy(links_np.astype(np.float32)).cuda()
    hist_out = torch.zeros_like(hist)
    links_out = torch.empty((B, ell, wl.d), dtype=torch.float32, device="cuda")
    Bd.lime_xor_layer(L.ctx, 0, hist, off, B, links32, shared_links, hist_out, links_out, L.workspace(B, total))
    assert Bd.lime_device_status(L.ctx) == 0
    cfg = Hh.oracle_config(wl, phi=O.SILU)
    lw = Hh.oracle_layers(inp, wl)[0]
    table64 = synth.storage_to_f64(inp["table"], wl.dtype)
    offh = O.lengths_to_offsets(lengths)
    for b in range(B):
        E = O.gather_history(table64, inp["hist_ids"][offh[b]:offh[b + 1]])
        S_next, T_next = O.xor_layer(E, links_np[b], lw, cfg)
        assert np.abs(Hh.to_f64(links_out[b]) - T_next).max() <= 4e-2 * max(1.0, np.abs(T_next).max()), b
        # unscaled scores through SiLU are not bounded like softmax weights, so single elements err more; the mean
        # error must still be a fraction of a per cent of the spread (a wrong divisor or a dropped chunk is not)
        assert np.abs(Hh.to_f64(links_out[b]) - T_next).mean() <= 1e-2 * max(T_next.std(), 1e-6) + 1e-5, b
        if lengths[b]:
            got = Hh.to_f64(hist_out[offh[b]:offh[b + 1]])
            assert np.abs(got - S_next).max() <= 4e-2 * max(1.0, np.abs(S_next).max()), (b, np.abs(got - S_next).max())
            assert np.abs(got - S_next).mean() <= 1e-2 * max(S_next.std(), 1e-6) + 1e-5, (b, np.abs(got - S_next).mean())


@pytest.mark.parametrize("H", [8, 4, 2])
@pytest.mark.parametrize("lengths", [[1], [63, 64, 65, 127, 128, 129], [0, 300, 5, 0, 1000], [256] * 40, [4095, 513, 4097, 9000]])
@pytest.mark.parametrize("shared_links", [True, False])
@pytest.mark.parametrize("phi", ["softmax", "silu"])
def test_xor_layer_tensor_core_path_d256(H, lengths, shared_links, phi):
    """One XOR layer at d = d_ff = 256 with 64 links (the shape of `production_ragged`: H = 8; also 4 and 2 heads) on the
    kernels built for that width: ragged histories around the 64-token tile of the link attention, the 128-token tile
    of the history update and the chunk length (several chunks per user, merged partials), shared and per-user link
    rows, softmax and the SiLU form of Algorithms 1-2.  The rows go in raw, so the library normalises them first."""
    Bd = _lib()
    B, ell, d = len(lengths), 64, 256
    silu = phi == "silu"
    wl = small(synth.BF16, B=B, n_min=0, n_max=1, d=d, H=H, ell=ell, n_layers=1, V=3000, table_std=0.05)
    inp = synth.make_inputs(wl, seed=H + B)
    inp["lengths"] = np.asarray(lengths, dtype=np.int32)
    total = int(sum(lengths))
    inp["hist_ids"] = synth.zipf_ids(3, "h", total, wl.V, 1.1)
    dev = Hh.DeviceBatch(wl, inp, phi=Bd.LIME_PHI_SILU if silu else Bd.LIME_PHI_SOFTMAX)
    L = dev.lime
    off = L.lengths_to_offsets(dev.lengths)
    hist = L.gather_history(dev.table, dev.hist_ids)
    if shared_links:
        links_np = synth.storage_to_f64(inp["links"], wl.dtype)[None].repeat(B, axis=0)
        links32 = dev.links.float().contiguous()
    else:
        links_np = np.random.default_rng(9).normal(size=(B, ell, d)).astype(np.float32).astype(np.float64)
        links32 = torch.from_numpy(links_np.astype(np.float32)).cuda()
    hist_out = torch.zeros_like(hist)
    links_out = torch.empty((B, ell, d), dtype=torch.float32, device="cuda")
    Bd.lime_xor_layer(L.ctx, 0, hist, off, B, links32, shared_links, hist_out if total else None, links_out,
                      L.workspace(B, total))
    assert Bd.lime_device_status(L.ctx) == 0
    cfg = Hh.oracle_config(wl, phi=O.SILU if silu else O.SOFTMAX)
    lw = Hh.oracle_layers(inp, wl)[0]
    table64 = synth.storage_to_f64(inp["table"], wl.dtype)
    offh = O.lengths_to_offsets(lengths)
    for b in range(B):
        E = O.gather_history(table64, inp["hist_ids"][offh[b]:offh[b + 1]])
        S_next, T_next = O.xor_layer(E, links_np[b], lw, cfg)
        got_t = Hh.to_f64(links_out[b])
        assert np.abs(got_t - T_next).max() <= 4e-2 * max(1.0, np.abs(T_next).max()), (b, np.abs(got_t - T_next).max())
        assert np.abs(got_t - T_next).mean() <= 1e-2 * max(T_next.std(), 1e-6) + 1e-5, (b, np.abs(got_t - T_next).mean())
        if lengths[b]:
            got = Hh.to_f64(hist_out[offh[b]:offh[b + 1]])
            assert np.abs(got - S_next).max() <= 4e-2 * max(1.0, np.abs(S_next).max()), (b, np.abs(got - S_next).max())
            assert np.abs(got - S_next).mean() <= 1e-2 * max(S_next.std(), 1e-6) + 1e-5, (b, np.abs(got - S_next).mean())


def test_config2_bf16_baseline_silu_sampled():
    # the bench workload with the SiLU form of the attention, through the fused lookup + LayerNorm as bench.py runs it
    wl = synth.named_workloads()["bf16_baseline"].replace(B=64)
    inp = synth.make_inputs(wl, seed=3)
    Bd = _lib()
    out = Hh.DeviceBatch(wl, inp, phi=Bd.LIME_PHI_SILU).run(normalized=True)
    torch.cuda.synchronize()
    cfg, layers = Hh.oracle_config(wl, phi=O.SILU), Hh.oracle_layers(inp, wl)
    table64 = synth.storage_to_f64(inp["table"], wl.dtype)
    links64 = synth.storage_to_f64(inp["links"], wl.dtype)
    off = O.lengths_to_offsets(inp["lengths"])
    r = np.random.default_rng(3)
    got_all, want_all = [], []
    for b in [0, 31, 63]:
        rows = np.sort(r.choice(wl.C, size=64, replace=False))
        lg, _, _ = Hh.oracle_user(inp, wl, b, off, table64, links64, layers, cfg, cand_rows=rows)
        got_all.append(Hh.to_f64(out["logits"][b * wl.C:(b + 1) * wl.C])[rows])
        want_all.append(lg)
    _check_logits(np.concatenate(got_all), np.concatenate(want_all), wl.dtype)


@pytest.mark.parametrize("d,H,ell,dtype", [(128, 4, 32, synth.BF16), (128, 4, 64, synth.BF16), (256, 8, 64, synth.BF16),
                                           (32, 2, 8, synth.F32), (64, 2, 33, synth.BF16)])
def test_xor_layer_in_place(d, H, ell, dtype):
    """hist_out may alias hist_in: the layer call with the history updated in place gives the same rows and link rows
    as the call with a separate output, on the tensor-core shapes and on the generic path."""
    Bd = _lib()
    lengths = [130, 0, 515, 64]
    B = len(lengths)
    wl = small(dtype, B=B, n_min=0, n_max=1, d=d, H=H, ell=ell, n_layers=1, V=3000, table_std=0.05 if dtype == synth.BF16 else 1.0)
    inp = synth.make_inputs(wl, seed=d + ell)
    inp["lengths"] = np.asarray(lengths, dtype=np.int32)
    total = int(sum(lengths))
    inp["hist_ids"] = synth.zipf_ids(3, "h", total, wl.V, 1.1)
    dev = Hh.DeviceBatch(wl, inp)
    L = dev.lime
    off = L.lengths_to_offsets(dev.lengths)
    hist = L.gather_history(dev.table, dev.hist_ids)
    links32 = dev.links.float().contiguous()
    ws = L.workspace(B, total)
    sep_hist, sep_links = torch.zeros_like(hist), torch.empty((B, ell, d), dtype=torch.float32, device="cuda")
    Bd.lime_xor_layer(L.ctx, 0, hist, off, B, links32, True, sep_hist, sep_links, ws)
    inp_hist, inp_links = hist.clone(), torch.empty_like(sep_links)
    Bd.lime_xor_layer(L.ctx, 0, inp_hist, off, B, links32, True, inp_hist, inp_links, ws)
    assert Bd.lime_device_status(L.ctx) == 0
    assert torch.equal(inp_hist, sep_hist)
    assert torch.equal(inp_links, sep_links)
    # and the separate-output call matches the oracle
    cfg, lw = Hh.oracle_config(wl), Hh.oracle_layers(inp, wl)[0]
    table64, links64 = synth.storage_to_f64(inp["table"], dtype), synth.storage_to_f64(inp["links"], dtype)
    offh = O.lengths_to_offsets(lengths)
    tol = 2e-4 if dtype == synth.F32 else 4e-2
    for b in range(B):
        S_next, T_next = O.xor_layer(O.gather_history(table64, inp["hist_ids"][offh[b]:offh[b + 1]]), links64, lw, cfg)
        assert np.abs(Hh.to_f64(sep_links[b]) - T_next).max() <= tol * max(1.0, np.abs(T_next).max())
        if lengths[b]:
            assert np.abs(Hh.to_f64(sep_hist[offh[b]:offh[b + 1]]) - S_next).max() <= tol * max(1.0, np.abs(S_next).max())


@pytest.mark.parametrize("ell,H", [(32, 4), (64, 4)])
def test_xor_layer_tensor_core_path_many_users(ell, H):
    """More users than the kernels stage offsets for in shared memory (1024): the work lists are then read from global
    memory.  Short ragged histories (some empty, some longer than a tile), sampled users checked against the oracle."""
    Bd = _lib()
    B = 1100
    r = np.random.default_rng(5)
    lengths = r.integers(0, 200, size=B).astype(np.int32)
    lengths[[0, 7, 500, 1099]] = [130, 0, 257, 129]
    wl = small(synth.BF16, B=B, n_min=0, n_max=1, d=128, H=H, ell=ell, n_layers=1, V=3000, table_std=0.05)
    inp = synth.make_inputs(wl, seed=ell)
    inp["lengths"] = lengths
    total = int(lengths.sum())
    inp["hist_ids"] = synth.zipf_ids(4, "h", total, wl.V, 1.1)
    dev = Hh.DeviceBatch(wl, inp)
    L = dev.lime
    off = L.lengths_to_offsets(dev.lengths)
    hist = L.gather_history(dev.table, dev.hist_ids)
    links32 = dev.links.float().contiguous()
    hist_out = torch.zeros_like(hist)
    links_out = torch.empty((B, ell, wl.d), dtype=torch.float32, device="cuda")
    Bd.lime_xor_layer(L.ctx, 0, hist, off, B, links32, True, hist_out, links_out, L.workspace(B, total))
    assert Bd.lime_device_status(L.ctx) == 0
    cfg = Hh.oracle_config(wl)
    lw = Hh.oracle_layers(inp, wl)[0]
    table64 = synth.storage_to_f64(inp["table"], wl.dtype)
    links64 = synth.storage_to_f64(inp["links"], wl.dtype)
    offh = O.lengths_to_offsets(lengths)
    assert np.array_equal(off.cpu().numpy(), offh)
    for b in [0, 1, 7, 8, 499, 500, 501, 1023, 1024, 1025, 1098, 1099]:
        E = O.gather_history(table64, inp["hist_ids"][offh[b]:offh[b + 1]])
        S_next, T_next = O.xor_layer(E, links64, lw, cfg)
        assert np.abs(Hh.to_f64(links_out[b]) - T_next).max() <= 4e-2 * max(1.0, np.abs(T_next).max()), b
        if lengths[b]:
            got = Hh.to_f64(hist_out[offh[b]:offh[b + 1]])
            assert np.abs(got - S_next).max() <= 4e-2 * max(1.0, np.abs(S_next).max()), (b, np.abs(got - S_next).max())


@pytest.mark.parametrize("ln", [True, False])
def test_link_attention_running_max_is_raised_mid_history(ln):
    """History whose later tiles score far higher than the first one for half of the link rows (the second 128 tokens
    are the negated first 128, so every score flips sign), with a large softmax scale: the online softmax of the
    tensor-core kernel must raise its reference maximum and rescale its accumulator, and still match the oracle."""
    Bd = _lib()
    n, d, ell, H = 128 * 3 + 37, 128, 32, 4
    wl = small(synth.BF16, B=2, n_min=n, n_max=n, d=d, H=H, ell=ell, n_layers=1, V=2 * n, table_std=1.0)
    inp = synth.make_inputs(wl, seed=21)
    r = np.random.default_rng(21)
    base = r.normal(size=(1, d))
    rows = np.concatenate([base + 0.05 * r.normal(size=(128, d)), -base + 0.05 * r.normal(size=(128, d)),
                           r.normal(size=(n - 256, d))])
    table = np.concatenate([rows, rows[::-1]])                # user 1 sees the same tokens in reverse order
    inp["table"] = synth.to_storage(table, synth.BF16)
    inp["hist_ids"] = np.arange(2 * n, dtype=np.int32)
    scale = 1.0
    dev = Hh.DeviceBatch(wl, inp, ln=ln, attn_scale=scale)
    L = dev.lime
    off = L.lengths_to_offsets(dev.lengths)
    hist = L.gather_history(dev.table, dev.hist_ids)
    links_out = torch.empty((2, ell, d), dtype=torch.float32, device="cuda")
    Bd.lime_xor_layer(L.ctx, 0, hist, off, 2, dev.links.float().contiguous(), True, None, links_out, L.workspace(2, 2 * n))
    assert Bd.lime_device_status(L.ctx) == 0
    cfg = Hh.oracle_config(wl, ln=ln, attn_scale=scale)
    lw = Hh.oracle_layers(inp, wl)[0]
    table64, links64 = synth.storage_to_f64(inp["table"], synth.BF16), synth.storage_to_f64(inp["links"], synth.BF16)
    outs = []
    for b in range(2):
        E = table64[b * n:(b + 1) * n]
        # the flip really produces large jumps of the per-row maximum between the first two tiles
        Xn = O.layer_norm(E) if ln else E
        sc = ((O.layer_norm(links64) if ln else links64) @ lw["Wq"])[:, :d // H] @ (Xn @ lw["Wk"])[:, :d // H].T * scale
        if b == 0:
            assert (sc[:, 128:256].max(axis=1) - sc[:, :128].max(axis=1) > 8).sum() >= 4
        _, T_next = O.xor_layer(E, links64, lw, cfg, need_history=False)
        got = Hh.to_f64(links_out[b])
        assert np.abs(got - T_next).max() <= 4e-2 * max(1.0, np.abs(T_next).max()), np.abs(got - T_next).max()
        outs.append(got)
    # same multiset of tokens in another order: same result up to rounding (no positional term)
    assert np.abs(outs[0] - outs[1]).max() <= 4e-2 * max(1.0, np.abs(outs[0]).max())


@pytest.mark.parametrize("dtype", [synth.F32, synth.BF16])
@pytest.mark.parametrize("ell,d,H", [(1, 8, 1), (8, 64, 2), (32, 128, 4), (64, 128, 4), (64, 256, 8), (33, 40, 5)])
def test_encode_and_score_shapes(dtype, ell, d, H):
    wl = small(dtype, B=3, n_min=5, n_max=150, d=d, H=H, ell=ell, n_layers=2, C=40, V=700, table_std=0.5)
    inp = synth.make_inputs(wl, seed=ell + d)
    out = Hh.DeviceBatch(wl, inp).run()
    want_logits, want_ls = _oracle_batch(wl, inp)
    assert np.array_equal(out["off"].cpu().numpy(), O.lengths_to_offsets(inp["lengths"]))
    ls_tol = 2e-4 if dtype == synth.F32 else 5e-2
    assert np.abs(Hh.to_f64(out["link_states"]) - want_ls).max() <= ls_tol * max(1.0, np.abs(want_ls).max())
    _check_logits(Hh.to_f64(out["logits"]), want_logits, dtype, stress=True)


@pytest.mark.parametrize("phi,ln,gated", [(O.SOFTMAX, False, False), (O.SILU, True, True), (O.SILU, False, False),
                                          (O.SOFTMAX, True, False)])
def test_profiles_core_and_silu(phi, ln, gated):
    Bd = _lib()
    wl = small(synth.F32, B=2, n_min=0, n_max=90, n_layers=3, table_std=0.7)
    inp = synth.make_inputs(wl, seed=5)
    inp["lengths"][0] = 0                                   # an empty history in the batch
    inp["hist_ids"] = inp["hist_ids"][: int(inp["lengths"].sum())]
    dev = Hh.DeviceBatch(wl, inp, phi=Bd.LIME_PHI_SILU if phi == O.SILU else Bd.LIME_PHI_SOFTMAX, ln=ln, gated_mlp=gated)
    out = dev.run()
    want_logits, want_ls = _oracle_batch(wl, inp, phi=phi, ln=ln, gated_mlp=gated)
    assert np.abs(Hh.to_f64(out["link_states"]) - want_ls).max() <= 2e-4 * max(1.0, np.abs(want_ls).max())
    _check_logits(Hh.to_f64(out["logits"]), want_logits, synth.F32)


def test_candidate_side_projections_and_link_context():
    Bd = _lib()
    wl = small(synth.F32, B=2, n_min=30, n_max=60, n_layers=2)
    inp = synth.make_inputs(wl, seed=6)
    cand_np = {k: synth.normal_storage(6, "c" + k, (wl.d, wl.d), wl.d ** -0.5, wl.dtype) for k in ("Wq", "Wk", "Wv")}
    out = Hh.DeviceBatch(wl, inp, cand=cand_np).run()
    want_logits, want_ls = _oracle_batch(wl, inp, cand_np=cand_np)
    assert np.abs(Hh.to_f64(out["link_states"]) - want_ls).max() <= 2e-4 * max(1.0, np.abs(want_ls).max())
    _check_logits(Hh.to_f64(out["logits"]), want_logits, synth.F32)
    # per-user contextualised links L^C (Eq. 2's output) instead of the shared L
    dev = Hh.DeviceBatch(wl, inp)
    LC = synth.normal_storage(7, "lc", (wl.B, wl.ell, wl.d), 1.0, synth.F32)
    off = dev.lime.lengths_to_offsets(dev.lengths)
    hist = dev.lime.gather_history(dev.table, dev.hist_ids)
    ls = dev.lime.encode_user(hist, off, torch.from_numpy(LC).cuda())
    cfg, layers = Hh.oracle_config(wl), Hh.oracle_layers(inp, wl)
    table64 = synth.storage_to_f64(inp["table"], wl.dtype)
    offh = O.lengths_to_offsets(inp["lengths"])
    for b in range(wl.B):
        E = O.gather_history(table64, inp["hist_ids"][offh[b]:offh[b + 1]])
        LP, _ = O.encode_user(E, LC[b].astype(np.float64), layers, cfg)
        assert np.abs(Hh.to_f64(ls[b]) - LP).max() <= 2e-4 * max(1.0, np.abs(LP).max())


@pytest.mark.parametrize("dtype,d,H,ell,proj", [(synth.F32, 32, 2, 8, False), (synth.F32, 64, 4, 5, True),
                                                 (synth.BF16, 128, 4, 32, False), (synth.BF16, 128, 8, 16, True),
                                                 (synth.BF16, 128, 2, 32, False), (synth.BF16, 128, 4, 64, False),
                                                 (synth.BF16, 64, 2, 33, False)])
def test_candidate_side_head_by_head(dtype, d, H, ell, proj):
    """Eq. 1 applied to Eq. 4 head by head (cand_heads = H): cached weights [C x H x ell], link states expanded per head,
    logits against the oracle's per-head form.  H * ell = 128 runs the tensor-core precompute (per-head softmax groups)
    and scorer; 256 and odd sizes the generic kernels."""
    Bd = _lib()
    wl = small(dtype, B=3, n_min=20, n_max=200, d=d, H=H, ell=ell, n_layers=2, C=300, V=2000,
               table_std=0.05 if dtype == synth.BF16 else 1.0)
    inp = synth.make_inputs(wl, seed=d + ell)
    cand_np = None
    if proj:
        cand_np = {k: synth.normal_storage(6, "c" + k, (d, d), d ** -0.5, dtype) for k in ("Wq", "Wk", "Wv")}
    dev = Hh.DeviceBatch(wl, inp, cand=cand_np, cand_heads=H)
    out = dev.run()
    assert tuple(out["W"].shape) == (wl.B * wl.C, H * ell) and tuple(out["link_states"].shape) == (wl.B, H * ell, d)
    cfg, layers = Hh.oracle_config(wl), Hh.oracle_layers(inp, wl)
    table64 = synth.storage_to_f64(inp["table"], dtype)
    links64 = synth.storage_to_f64(inp["links"], dtype)
    cw = {k + "_c": synth.storage_to_f64(v, dtype) for k, v in cand_np.items()} if cand_np else None
    off = O.lengths_to_offsets(inp["lengths"])
    got_all, want_all = [], []
    for b in range(wl.B):
        lg, LS, W = Hh.oracle_user(inp, wl, b, off, table64, links64, layers, cfg, cand_w=cw, cand_heads=True)
        got_w = Hh.to_f64(out["W"][b * wl.C:(b + 1) * wl.C]).reshape(wl.C, H, ell)
        assert np.abs(got_w.sum(axis=2) - 1.0).max() <= (1e-5 if dtype == synth.F32 else 2e-2)
        assert np.abs(got_w - W).max() <= (1e-5 if dtype == synth.F32 else 2.0 ** -8)
        got_all.append(Hh.to_f64(out["logits"][b * wl.C:(b + 1) * wl.C]))
        want_all.append(lg)
    _check_logits(np.concatenate(got_all), np.concatenate(want_all), dtype, stress=True)


# ----------------------------------------------------------------------------- the named workloads
def test_config1_tiny_fp32_full_parity():
    wl = synth.named_workloads()["tiny_fp32"]
    inp = synth.make_inputs(wl, seed=0)
    out = Hh.DeviceBatch(wl, inp).run()
    want_logits, want_ls = _oracle_batch(wl, inp)
    got = Hh.to_f64(out["logits"])
    assert got.shape == (wl.B * wl.C,)
    _check_logits(got, want_logits, synth.F32)
    assert np.abs(got - want_logits).max() <= 1e-3 * want_logits.std()     # fp32 path is far inside 1e-4


def _sampled_parity(wl, seed, users, n_cand=64, normalized=False):
    inp = synth.make_inputs(wl, seed=seed)
    out = Hh.DeviceBatch(wl, inp).run(normalized=normalized)
    torch.cuda.synchronize()
    cfg, layers = Hh.oracle_config(wl), Hh.oracle_layers(inp, wl)
    table64 = synth.storage_to_f64(inp["table"], wl.dtype)
    links64 = synth.storage_to_f64(inp["links"], wl.dtype)
    off = O.lengths_to_offsets(inp["lengths"])
    assert np.array_equal(out["off"].cpu().numpy(), off)
    # gathered rows: bit exact on a sample of tokens
    r = np.random.default_rng(seed)
    tok = r.integers(0, off[-1], size=512)
    if normalized:
        # rows after the fused lookup + LayerNorm: the oracle's LayerNorm of the same table rows, to bf16 rounding
        got_rows = Hh.to_f64(out["hist"][torch.from_numpy(tok).cuda()])
        want_rows = O.layer_norm(table64[inp["hist_ids"][tok]])
        assert np.abs(got_rows - want_rows).max() <= 2.0 ** -8 * max(1.0, np.abs(want_rows).max())
    else:
        got_rows = out["hist"][torch.from_numpy(tok).cuda()].view(torch.int16).cpu().numpy().view(np.uint16)
        assert np.array_equal(got_rows, inp["table"][inp["hist_ids"][tok]])
    got_all, want_all = [], []
    for b in users:
        rows = np.sort(r.choice(wl.C, size=min(n_cand, wl.C), replace=False))
        lg, _, _ = Hh.oracle_user(inp, wl, b, off, table64, links64, layers, cfg, cand_rows=rows)
        got_all.append(Hh.to_f64(out["logits"][b * wl.C:(b + 1) * wl.C])[rows])
        want_all.append(lg)
    _check_logits(np.concatenate(got_all), np.concatenate(want_all), wl.dtype)


def test_config2_bf16_baseline_sampled():
    wl = synth.named_workloads()["bf16_baseline"]
    _sampled_parity(wl, seed=0, users=[0, 1, 100, 255])


@pytest.mark.parametrize("normalized", [False, True])
def test_config2_bf16_baseline_every_logit(normalized):
    """The workload bench.py times, in its launch shape, all 256 users x 2048 candidates against the oracle, for both call
    sequences (raw rows; rows normalised by the lookup, which is what the bench runs)."""
    wl = synth.named_workloads()["bf16_baseline"]
    inp = synth.make_inputs(wl, seed=5)
    out = Hh.DeviceBatch(wl, inp).run(normalized=normalized)
    torch.cuda.synchronize()
    want, _ = _oracle_batch(wl, inp)
    got = Hh.to_f64(out["logits"])
    assert got.shape == want.shape == (wl.B * wl.C,)
    _check_logits(got, want, wl.dtype)
    # no user stands out: the per-user worst error obeys the same relative bound
    per_user = np.abs(got - want).reshape(wl.B, wl.C).max(axis=1)
    assert per_user.max() <= REL_BF16 * want.std() + 1e-4, int(np.argmax(per_user))


def test_config2_step_replayed_from_a_cuda_graph_matches_the_eager_run():
    """The bench workload's step (offsets -> lookup + LayerNorm -> encode -> score) captured once into a CUDA graph and
    replayed back to back, as bench.py times it: in a replay the kernels follow one another without the host between
    them, and those launched for programmatic dependent launch start their set-up while the previous kernel still
    runs.  Every replay must give the eager run's logits bit for bit (the kernels are deterministic), and the eager run
    is checked against the oracle on a few users."""
    wl = synth.named_workloads()["bf16_baseline"]
    inp = synth.make_inputs(wl, seed=7)
    db = Hh.DeviceBatch(wl, inp)
    L = db.lime

    def step():
        off = L.lengths_to_offsets(db.lengths)
        hist = L.gather_history_normalized(db.table, db.hist_ids)
        ls = L.encode_user_normalized(hist, off)
        return L.score_candidates(ls, W, cand, C=wl.C)

    cand = L.gather_history(db.table, db.cand_ids)
    W = L.precompute_candidate_links(cand)
    eager = step().clone()
    db.Bd.lime_device_status(L.ctx)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        for _ in range(2):
            step()                                   # warm-up on the capture stream: sizes shared-memory attributes
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        out = step()
    for _ in range(25):
        g.replay()
    torch.cuda.synchronize()
    db.Bd.lime_device_status(L.ctx)
    assert torch.equal(out, eager)
    # between replays, with the output cleared: a kernel that ran ahead of its input would leave zeros or stale rows
    for _ in range(5):
        out.zero_()
        g.replay()
        g.replay()
        torch.cuda.synchronize()
        assert torch.equal(out, eager)
    off = O.lengths_to_offsets(inp["lengths"])
    table64, links64 = Hh.LazyTable64(inp["table"], wl.dtype), synth.storage_to_f64(inp["links"], wl.dtype)
    cfg, layers = Hh.oracle_config(wl), Hh.oracle_layers(inp, wl)
    got = Hh.to_f64(eager).reshape(wl.B, wl.C)
    for b in (0, 77, 255):
        want = Hh.oracle_user(inp, wl, b, off, table64, links64, layers, cfg)[0]
        _check_logits(got[b], want, wl.dtype)


def test_config2_bf16_baseline_normalized_lookup_sampled():
    # the launch sequence bench.py times: lookup fused with the first layer's LayerNorm, encode on normalised rows
    wl = synth.named_workloads()["bf16_baseline"]
    _sampled_parity(wl, seed=2, users=[0, 3, 128, 255], normalized=True)


@pytest.mark.parametrize("name,kw", [("tiny_fp32", {}), ("long_history", dict(n_min=700, n_max=1500, B=6)),
                                     ("production_ragged", dict(B=8, V=50_000, C=256, n_min=100, n_max=700))])
def test_normalized_lookup_on_other_paths(name, kw):
    # fp32 storage and d = 256 run the generic path, which normalises again (a fixed point up to rounding);
    # H * ell = 256 runs the streamed-operand kernels without their LayerNorm
    wl = synth.named_workloads()[name].replace(**kw) if kw else synth.named_workloads()[name]
    _sampled_parity_any_dtype(wl, normalized=True)


def _sampled_parity_any_dtype(wl, normalized):
    inp = synth.make_inputs(wl, seed=4)
    out = Hh.DeviceBatch(wl, inp).run(normalized=normalized)
    torch.cuda.synchronize()
    cfg, layers = Hh.oracle_config(wl), Hh.oracle_layers(inp, wl)
    table64 = synth.storage_to_f64(inp["table"], wl.dtype)
    links64 = synth.storage_to_f64(inp["links"], wl.dtype)
    off = O.lengths_to_offsets(inp["lengths"])
    got_all, want_all = [], []
    for b in sorted({0, wl.B - 1}):
        lg, _, _ = Hh.oracle_user(inp, wl, b, off, table64, links64, layers, cfg)
        got_all.append(Hh.to_f64(out["logits"][b * wl.C:(b + 1) * wl.C]))
        want_all.append(lg)
    _check_logits(np.concatenate(got_all), np.concatenate(want_all), wl.dtype)


@pytest.mark.parametrize("seed", list(range(11, 41)))
def test_random_ragged_batches_on_the_tensor_core_path(seed):
    """Randomly drawn batch shapes (users, ragged lengths around tile and chunk boundaries, empty histories, layers,
    heads x links, softmax or SiLU): both call sequences (raw rows, rows normalised by the lookup) must agree with each
    other, and sampled users with the oracle."""
    Bd = _lib()
    r = np.random.default_rng(seed)
    ell, H = [(32, 4), (16, 8), (64, 4), (32, 8), (64, 8)][seed % 5]
    B = int(r.integers(1, 200))
    kinds = r.integers(0, 5, size=B)
    lengths = np.where(kinds == 0, 0,
              np.where(kinds == 1, r.integers(1, 128, size=B),
              np.where(kinds == 2, 128 * r.integers(1, 6, size=B) + r.integers(-1, 2, size=B),
              np.where(kinds == 3, 512 * r.integers(1, 4, size=B) + r.integers(-1, 2, size=B),
                       r.integers(1, 3000, size=B))))).astype(np.int32)
    n_layers = int(r.integers(1, 4))
    silu = bool(seed % 2)
    wl = small(synth.BF16, B=B, n_min=0, n_max=1, d=128, H=H, ell=ell, n_layers=n_layers, V=5000, C=96, table_std=0.05)
    inp = synth.make_inputs(wl, seed=seed)
    inp["lengths"] = lengths
    inp["hist_ids"] = synth.zipf_ids(seed, "h", int(lengths.sum()), wl.V, 1.1)
    phi = Bd.LIME_PHI_SILU if silu else Bd.LIME_PHI_SOFTMAX
    raw = Hh.DeviceBatch(wl, inp, phi=phi).run()
    nrm = Hh.DeviceBatch(wl, inp, phi=phi).run(normalized=True)
    a, b = Hh.to_f64(raw["logits"]), Hh.to_f64(nrm["logits"])
    assert np.isfinite(a).all() and np.isfinite(b).all()
    spread = max(a.std(), 1e-6)
    assert np.abs(a - b).max() <= 2 * TOL_BF16 * max(1.0, np.abs(a).max())
    assert np.abs(a - b).mean() <= 2e-2 * spread + 1e-5
    cfg = Hh.oracle_config(wl, phi=O.SILU if silu else O.SOFTMAX)
    layers = Hh.oracle_layers(inp, wl)
    table64 = synth.storage_to_f64(inp["table"], wl.dtype)
    links64 = synth.storage_to_f64(inp["links"], wl.dtype)
    off = O.lengths_to_offsets(lengths)
    users = sorted({0, B - 1, int(np.argmax(lengths)), int(np.argmin(lengths))})
    for out in (raw, nrm):
        got_all, want_all = [], []
        for u in users:
            lg, _, _ = Hh.oracle_user(inp, wl, u, off, table64, links64, layers, cfg)
            got_all.append(Hh.to_f64(out["logits"][u * wl.C:(u + 1) * wl.C]))
            want_all.append(lg)
        got, want = np.concatenate(got_all), np.concatenate(want_all)
        # max-abs against 2e-2 (scaled by max|logit| where the drawn shape gives logits beyond one: SiLU weights are not
        # normalised, so stacked layers grow) and against 10 % of the spread; the mean error against 2 % of it
        _check_logits(got, want, wl.dtype, stress=True, rel=REL_BF16_DRAWN)
        assert np.abs(got - want).mean() <= 2e-2 * max(want.std(), 1e-6) + 1e-5


def test_config3_candidate_sweep_sampled():
    wl = synth.named_workloads()["candidate_sweep"].replace(C=4096)
    _sampled_parity(wl, seed=0, users=[0, 63])


def test_config4_long_history_sampled():
    wl = synth.named_workloads()["long_history"].replace(n_min=4096, n_max=4096, B=8)
    _sampled_parity(wl, seed=0, users=[0, 7])


def test_config3_candidate_sweep_largest_C_sampled():
    # the last point of the candidate sweep (App. F): 32768 candidates per user, in the launch shape the bench times
    wl = synth.named_workloads()["candidate_sweep"].replace(C=32768)
    _sampled_parity(wl, seed=1, users=[0, 31, 63], n_cand=48)


def test_config4_long_history_longest_N_sampled():
    # the last point of the history sweep: 32768 tokens per user, 32 users (many chunks per user, merged partials)
    wl = synth.named_workloads()["long_history"].replace(n_min=32768, n_max=32768)
    _sampled_parity(wl, seed=1, users=[0, 31], n_cand=48)


def test_config5_production_ragged_full_size_sampled():
    """`production_ragged` at its named size - 1024 users with 1024..4096 history items each (2.6 M tokens), d = 256,
    8 heads, 64 links, 4 layers, 8192 candidates per user from a 4M x 256 table - through the call sequence bench.py
    times (lookup fused with the first LayerNorm, encode on normalised rows, dense scorer) and, for the candidates, also
    by id from the corpus caches.  Offsets bit exact; sampled gathered rows against the oracle's LayerNorm of the table
    rows; the users with the shortest and the longest history, the first and the last, each on 48 sampled candidates,
    against the oracle."""
    Bd = _lib()
    wl = synth.named_workloads()["production_ragged"]
    inp = synth.make_inputs(wl, seed=0)
    dev = Hh.DeviceBatch(wl, inp)
    out = dev.run(normalized=True)
    torch.cuda.synchronize()
    off = O.lengths_to_offsets(inp["lengths"])
    assert np.array_equal(out["off"].cpu().numpy(), off)
    table64 = Hh.LazyTable64(inp["table"], wl.dtype)
    links64 = synth.storage_to_f64(inp["links"], wl.dtype)
    cfg, layers = Hh.oracle_config(wl), Hh.oracle_layers(inp, wl)
    r = np.random.default_rng(0)
    tok = r.integers(0, off[-1], size=256)
    got_rows = Hh.to_f64(out["hist"][torch.from_numpy(tok).cuda()])
    want_rows = O.layer_norm(O.gather_history(table64, inp["hist_ids"][tok]))
    assert np.abs(got_rows - want_rows).max() <= 2.0 ** -8 * max(1.0, np.abs(want_rows).max())
    # the same candidates scored by id straight from the corpus caches (weights of the whole table precomputed once)
    w_corpus = dev.lime.precompute_candidate_links(dev.table)
    by_id = dev.lime.score_candidates(out["link_states"], w_corpus, dev.table, C=wl.C, cand_ids=dev.cand_ids,
                                      total_cands=wl.B * wl.C)
    assert Bd.lime_device_status(dev.lime.ctx) == 0
    users = sorted({int(np.argmin(inp["lengths"])), int(np.argmax(inp["lengths"])), 0, wl.B - 1})
    got_all, got_id, want_all = [], [], []
    for b in users:
        rows = np.sort(r.choice(wl.C, size=48, replace=False))
        lg, _, _ = Hh.oracle_user(inp, wl, b, off, table64, links64, layers, cfg, cand_rows=rows)
        got_all.append(Hh.to_f64(out["logits"][b * wl.C:(b + 1) * wl.C])[rows])
        got_id.append(Hh.to_f64(by_id[b * wl.C:(b + 1) * wl.C])[rows])
        want_all.append(lg)
    _check_logits(np.concatenate(got_all), np.concatenate(want_all), wl.dtype)
    _check_logits(np.concatenate(got_id), np.concatenate(want_all), wl.dtype)
    assert torch.isfinite(out["logits"]).all()


def test_config5_production_ragged_sampled():
    wl = synth.named_workloads()["production_ragged"].replace(B=32, V=200_000, C=512)
    inp_len = synth.history_lengths(0, wl.B, wl.n_min, wl.n_max)
    users = [int(np.argmin(inp_len)), int(np.argmax(inp_len))]
    _sampled_parity(wl, seed=0, users=users)

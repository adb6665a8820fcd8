"""Parity of the two feed-forward networks (Eq. 2's link contextualisation; the interaction network of Sec. 3.3)
against the fp64 oracle, through the C ABI.  Tolerances: fp32 storage 1e-4 (relative to the largest logit); bf16
storage 2e-2 absolute and 3e-2 of the spread of the oracle's logits (one extra bf16 rounding, of the per-user product
link_states . W_0[:d], on top of the stored operands)."""
import numpy as np
import pytest
import torch

from oracle import lime_oracle as O
from paper_2510_18239_b200 import synth
from tests import lime_helpers as Hh

pytestmark = [pytest.mark.gpu, pytest.mark.skipif(not torch.cuda.is_available(), reason="needs a CUDA device")]

REL_HEAD_BF16 = 3e-2


def _lib():
    from paper_2510_18239_b200 import binding
    return binding


def _ffn64(layers, dtype):
    return [(synth.storage_to_f64(W, dtype), b.astype(np.float64)) for W, b in layers]


def _dev_ffn(Bd, layers, dtype):
    return [(Bd.to_device(W, dtype), torch.from_numpy(b).cuda()) for W, b in layers]


def _head_case(seed, B, C, d, ell, dtype, w_rows=None):
    """Link states, cached weights (rows sum to 1) and candidate embeddings in storage format."""
    r = np.random.default_rng(seed)
    LS = synth.to_storage(r.normal(size=(B, ell, d)) * 0.5, dtype)
    n = B * C if w_rows is None else w_rows
    W = synth.to_storage(O.softmax_rows(r.normal(size=(n, ell)) * 1.5), dtype)
    T = synth.to_storage(r.normal(size=(n, d)) * 0.5, dtype)
    return LS, W, T


def _kernels_run(Bd, fn):
    Bd.lime_profile_start(64)
    out = fn()
    torch.cuda.synchronize()
    rec, _ = Bd.lime_profile_stop(64)
    return out, [k for k, _ in rec]


@pytest.mark.parametrize("d,ell,n1,B,C", [(128, 32, 96, 3, 300), (128, 64, 96, 2, 129), (256, 64, 96, 3, 200),
                                          (128, 128, 64, 2, 130), (64, 32, 16, 1, 5), (128, 32, 128, 2, 256),
                                          (128, 32, 96, 40, 1024), (256, 64, 96, 20, 2048)])
def test_interaction_head_on_tensor_cores(d, ell, n1, B, C):
    """One hidden layer, bf16, dense candidate streams: the tcgen05 scorer (weight rows and link-state products as
    64- / 128-byte swizzled operands; many tiles per CTA and several users per CTA in the last two cases)."""
    Bd = _lib()
    dtype = synth.BF16
    lime = Bd.Lime(d, 4, ell, 1, dtype=Bd.LIME_BF16)
    LS, W, T = _head_case(d + ell + n1 + C, B, C, d, ell, dtype)
    layers = synth.ffn_weights(5, "head", (2 * d, n1, 1), dtype)
    dev = _dev_ffn(Bd, layers, dtype)
    lime.set_head(dev)
    ls_d, w_d, t_d = Bd.to_device(LS, dtype), Bd.to_device(W, dtype), Bd.to_device(T, dtype)
    got, names = _kernels_run(Bd, lambda: lime.score_candidates_head(ls_d, w_d, t_d, C=C))
    Bd.lime_device_status(lime.ctx)
    assert "k_score_head_tc" in names, names
    got = Hh.to_f64(got)
    L64 = _ffn64(layers, dtype)
    LS64, W64, T64 = (synth.storage_to_f64(x, dtype) for x in (LS, W, T))
    users = range(B) if B * C <= 4096 else sorted({0, 1, B // 2, B - 1})
    worst, spread = 0.0, 0.0
    for b in users:
        sl = slice(b * C, (b + 1) * C)
        want = O.score_candidates_head(W64[sl], LS64[b], T64[sl], L64)
        worst = max(worst, float(np.abs(got[sl] - want).max()))
        spread = max(spread, float(want.std()))
    assert worst <= 2e-2 and worst <= REL_HEAD_BF16 * spread + 1e-3, (worst, spread)


@pytest.mark.parametrize("dtype,widths", [(synth.F32, (24,)), (synth.F32, (24, 12)), (synth.F32, (40, 16, 8)),
                                          (synth.BF16, (32, 16)), (synth.BF16, (100,))])
def test_interaction_head_generic_paths(dtype, widths):
    """fp32 storage, deeper networks, widths the tensor-core kernel does not take: dense fixed-C slots, ragged candidate
    lists and candidates taken by id from corpus caches (ids outside the caches score 0 and lower the flag)."""
    Bd = _lib()
    d, ell, B, C, V = 32, 8, 3, 37, 211
    lime = Bd.Lime(d, 2, ell, 1, dtype=Bd.LIME_F32 if dtype == synth.F32 else Bd.LIME_BF16)
    layers = synth.ffn_weights(6, "head", (2 * d,) + tuple(widths) + (1,), dtype)
    lime.set_head(_dev_ffn(Bd, layers, dtype))
    L64 = _ffn64(layers, dtype)
    tol = 1e-4 if dtype == synth.F32 else 2e-2

    # dense, fixed C
    LS, W, T = _head_case(1, B, C, d, ell, dtype)
    LS64, W64, T64 = (synth.storage_to_f64(x, dtype) for x in (LS, W, T))
    ls_d = Bd.to_device(LS, dtype)
    got = Hh.to_f64(lime.score_candidates_head(ls_d, Bd.to_device(W, dtype), Bd.to_device(T, dtype), C=C))
    want = np.concatenate([O.score_candidates_head(W64[b * C:(b + 1) * C], LS64[b], T64[b * C:(b + 1) * C], L64) for b in range(B)])
    assert np.abs(got - want).max() <= tol * max(1.0, np.abs(want).max())

    # ragged candidate lists (one user without candidates)
    counts = np.array([5, 0, 32], dtype=np.int32)
    coff = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
    tot = int(coff[-1])
    got = Hh.to_f64(lime.score_candidates_head(ls_d, Bd.to_device(W[:tot], dtype), Bd.to_device(T[:tot], dtype),
                                               cand_off=torch.from_numpy(coff).cuda(), total_cands=tot))
    want = np.concatenate([O.score_candidates_head(W64[coff[b]:coff[b + 1]], LS64[b], T64[coff[b]:coff[b + 1]], L64) for b in range(B)])
    assert np.abs(got - want).max() <= tol * max(1.0, np.abs(want).max())

    # by id from corpus caches
    _, Wc, Tc = _head_case(2, B, C, d, ell, dtype, w_rows=V)
    Wc64, Tc64 = synth.storage_to_f64(Wc, dtype), synth.storage_to_f64(Tc, dtype)
    ids = np.random.default_rng(3).integers(0, V, size=B * C).astype(np.int32)
    ids[7], ids[50], ids[90] = -1, V, 2 ** 31 - 1
    flag = torch.full((1,), 2 ** 31 - 1, dtype=torch.int32, device="cuda")
    got = Hh.to_f64(lime.score_candidates_head(ls_d, Bd.to_device(Wc, dtype), Bd.to_device(Tc, dtype), C=C,
                                               cand_ids=torch.from_numpy(ids).cuda(), dev_flag=flag))
    ok = (ids >= 0) & (ids < V)
    want = np.zeros(B * C)
    for b in range(B):
        sl = np.arange(b * C, (b + 1) * C)
        keep = sl[ok[sl]]
        want[keep] = O.score_candidates_head(Wc64[ids[keep]], LS64[b], Tc64[ids[keep]], L64)
    assert np.abs(got - want).max() <= tol * max(1.0, np.abs(want).max())
    assert np.all(got[~ok] == 0.0) and int(flag.item()) == 7
    Bd.lime_device_status(lime.ctx)


@pytest.mark.parametrize("dtype", [synth.F32, synth.BF16])
@pytest.mark.parametrize("hidden", [(), (16,), (24, 40)])
def test_link_contextualisation_mlp(dtype, hidden):
    """Eq. 2: per user L^C = MLP(L (+) E^C), every row against the oracle; then the rows drive the user side (Eq. 8)."""
    Bd = _lib()
    wl = synth.Workload("ctx", B=5, n_min=9, n_max=40, d=32, H=2, ell=11, n_layers=2, C=16, dtype=dtype, V=300,
                        zipf_s=1.1, table_std=1.0, link_std=1.0)
    d_c = 6
    inp = synth.make_inputs(wl, seed=3)
    dev = Hh.DeviceBatch(wl, inp)
    lime = dev.lime
    layers = synth.ffn_weights(7, "ctx", (wl.d + d_c,) + tuple(hidden) + (wl.d,), dtype)
    lime.set_context_mlp(d_c, _dev_ffn(Bd, layers, dtype))
    ec = synth.normal_storage(8, "ec", (wl.B, d_c), 1.0, dtype)
    lc = lime.contextualize_links(Bd.to_device(ec, dtype))
    assert lc.dtype == torch.float32 and tuple(lc.shape) == (wl.B, wl.ell, wl.d)
    L64, links64, ec64 = _ffn64(layers, dtype), synth.storage_to_f64(inp["links"], dtype), synth.storage_to_f64(ec, dtype)
    want = np.stack([O.contextualize_links(links64, ec64[b], L64) for b in range(wl.B)])
    got = Hh.to_f64(lc)
    assert np.abs(got - want).max() <= 2e-5 * max(1.0, np.abs(want).max())

    # the contextualised links as the link rows of the user side, end to end
    off = lime.lengths_to_offsets(dev.lengths)
    hist = lime.gather_history(dev.table, dev.hist_ids)
    ls = lime.encode_user(hist, off, link_ctx=lc)
    cfg, lay = Hh.oracle_config(wl), Hh.oracle_layers(inp, wl)
    table64 = synth.storage_to_f64(inp["table"], dtype)
    offs = O.lengths_to_offsets(inp["lengths"])
    for b in range(wl.B):
        E = O.gather_history(table64, inp["hist_ids"][offs[b]:offs[b + 1]])
        LP, _ = O.encode_user(E, Hh.to_f64(lc[b]), lay, cfg)
        err = np.abs(Hh.to_f64(ls[b]) - LP).max()
        assert err <= (1e-4 if dtype == synth.F32 else 6e-2) * max(1.0, np.abs(LP).max()), (b, err)
    Bd.lime_device_status(lime.ctx)


def test_ffn_calls_need_their_networks():
    Bd = _lib()
    lime = Bd.Lime(32, 2, 8, 1, dtype=Bd.LIME_F32)
    x = torch.zeros((2, 4), device="cuda")
    with pytest.raises(Bd.LimeError) as e:
        Bd.lime_contextualize_links(lime.ctx, x, 2, torch.zeros((2, 8, 32), device="cuda"))
    assert e.value.status == 5
    assert Bd.lime_head_workspace_bytes(lime.ctx, 4) == 0
    # the context MLP's first layer folds the links: set_weights first
    layers = _dev_ffn(Bd, synth.ffn_weights(1, "c", (36, 32), synth.F32), synth.F32)
    with pytest.raises(Bd.LimeError) as e:
        lime.set_context_mlp(4, layers)
    assert e.value.status == 5


def test_bounded_wait_expires_and_reports():
    """Failure detection without a fault: a wait nothing can satisfy gives up after its limit, the kernel returns, the
    status word carries the code, and the context keeps working."""
    import time
    Bd = _lib()
    lime = Bd.Lime(32, 2, 8, 1, dtype=Bd.LIME_F32)
    assert Bd.lime_device_status(lime.ctx) == 0
    t0 = time.time()
    Bd.lime_selftest_wait_expiry(lime.ctx, 1000)          # 1 ms
    with pytest.raises(Bd.LimeError) as e:
        Bd.lime_device_status(lime.ctx)
    assert time.time() - t0 < 5.0
    assert e.value.status == 6 and "wait code 200" in str(e.value)
    assert Bd.lime_device_status(lime.ctx) == 0           # reading the word clears it
    # the context and the device are still usable
    off = lime.lengths_to_offsets(torch.tensor([3, 0, 4], dtype=torch.int32, device="cuda"))
    assert off.cpu().tolist() == [0, 3, 3, 7]
    with pytest.raises(Bd.LimeError):
        Bd.lime_selftest_wait_expiry(lime.ctx, 0)


@pytest.mark.parametrize("dtype,d,H,ell,n1", [(synth.BF16, 128, 2, 16, 64), (synth.F32, 32, 2, 8, 24)])
def test_interaction_head_after_the_whole_path_with_head_wise_candidate_side(dtype, d, H, ell, n1):
    """offsets -> lookup -> XOR layers -> link states -> precompute -> interaction network, with the candidate side run
    head by head (H * ell weight columns per candidate, link states expanded per head): every logit against the oracle."""
    Bd = _lib()
    wl = synth.Workload("headwise", B=3, n_min=20, n_max=150, d=d, H=H, ell=ell, n_layers=2, C=70, dtype=dtype, V=900,
                        zipf_s=1.1, table_std=0.5, link_std=1.0)
    inp = synth.make_inputs(wl, seed=5)
    dev = Hh.DeviceBatch(wl, inp, cand_heads=H)
    lime = dev.lime
    layers = synth.ffn_weights(9, "head", (2 * d, n1, 1), dtype)
    lime.set_head(_dev_ffn(Bd, layers, dtype))
    off = lime.lengths_to_offsets(dev.lengths)
    ls = lime.encode_user(lime.gather_history(dev.table, dev.hist_ids), off)
    cand = lime.gather_history(dev.table, dev.cand_ids)
    W = lime.precompute_candidate_links(cand)
    assert tuple(W.shape) == (wl.B * wl.C, H * ell) and tuple(ls.shape) == (wl.B, H * ell, d)
    got = Hh.to_f64(lime.score_candidates_head(ls, W, cand, C=wl.C))
    Bd.lime_device_status(lime.ctx)
    cfg, lay, L64 = Hh.oracle_config(wl), Hh.oracle_layers(inp, wl), _ffn64(layers, dtype)
    table64, links64 = synth.storage_to_f64(inp["table"], dtype), synth.storage_to_f64(inp["links"], dtype)
    offs = O.lengths_to_offsets(inp["lengths"])
    worst, spread = 0.0, 0.0
    for b in range(wl.B):
        want, _, _ = Hh.oracle_user(inp, wl, b, offs, table64, links64, lay, cfg, cand_heads=True, head=L64)
        worst = max(worst, float(np.abs(got[b * wl.C:(b + 1) * wl.C] - want).max()))
        spread = max(spread, float(want.std()))
    if dtype == synth.F32:
        assert worst <= 1e-4 * max(1.0, spread), (worst, spread)
    else:
        assert worst <= 2e-2 and worst <= 6e-2 * spread + 1e-3, (worst, spread)

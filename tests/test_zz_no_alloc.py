"""The allocation-free precompute entry point, for hosts that must not allocate device memory while serving (a frozen
memory pool, or a framework that owns the allocator).  It must give what the context-based entry point gives, also on
a second call with different weights (its scratch is a fixed array shared by all calls and keeps old contents), and
must refuse shapes beyond its fixed scratch.  Collected last on purpose: a run that stops at the first failure has
then already run every other test."""
import numpy as np
import pytest
import torch

from oracle import lime_oracle as O
from paper_2510_18239_b200 import synth

pytestmark = [pytest.mark.gpu, pytest.mark.skipif(not torch.cuda.is_available(), reason="needs a CUDA device")]


def _both(Bd, dtype, ell, d, M, seed, proj):
    dt = Bd.LIME_F32 if dtype == synth.F32 else Bd.LIME_BF16
    links = Bd.to_device(synth.normal_storage(seed, "l", (ell, d), 1.0, dtype), dtype)
    cand = Bd.to_device(synth.normal_storage(seed, "c", (M, d), 1.0, dtype), dtype)
    wq = Bd.to_device(synth.normal_storage(seed, "q", (d, d), d ** -0.5, dtype), dtype) if proj else None
    wk = Bd.to_device(synth.normal_storage(seed, "k", (d, d), d ** -0.5, dtype), dtype) if proj else None
    lime = Bd.Lime(d, max(1, d // 128), ell, 1, dtype=dt, gated_mlp=False)
    lime.set_weights(links, [{}], {k: v for k, v in (("Wq", wq), ("Wk", wk)) if v is not None})
    want = lime.precompute_candidate_links(cand)
    got = torch.empty_like(want)               # the caller owns every buffer, the output included
    Bd.lime_precompute_candidate_links_noalloc(dt, d, ell, 0.0, links, wq, wk, cand, got)
    torch.cuda.synchronize()
    # the expected value proper: the oracle's candidate->link weights (Eq. 4) on the same stored inputs
    f64 = lambda t: None if t is None else t.float().cpu().numpy().astype(np.float64)
    oracle = O.precompute_candidate_links(f64(cand), f64(links), O.OracleConfig(d=d, H=1, ell=ell, n_layers=1), f64(wq), f64(wk))
    return got.float().cpu().numpy(), want.float().cpu().numpy(), oracle


@pytest.mark.parametrize("dtype", [synth.BF16, synth.F32])
def test_noalloc_precompute_matches_context_path_twice_in_a_row(dtype):
    from paper_2510_18239_b200 import binding as Bd
    tol = 2e-5 if dtype == synth.F32 else 4e-3      # the tolerances of the precompute parity test
    # first call: projections present, 32 links; second call straight after: other weights, fewer links, no
    # projections - stale scratch from the first call would show up here.  Every result is held against the oracle
    # first, and against the context-based entry point second.
    got1, want1, oracle1 = _both(Bd, dtype, 32, 128, 777, seed=11, proj=True)
    assert np.abs(got1 - oracle1).max() <= tol
    assert np.abs(got1 - want1).max() <= tol
    got2, want2, oracle2 = _both(Bd, dtype, 16, 64, 300, seed=12, proj=False)
    assert np.abs(got2 - oracle2).max() <= tol
    assert np.abs(got2 - want2).max() <= tol
    assert np.abs(got2.sum(axis=1) - 1.0).max() <= 1e-2
    # the largest supported shape
    got3, want3, oracle3 = _both(Bd, dtype, 64, 256, 129, seed=13, proj=True)
    assert np.abs(got3 - oracle3).max() <= tol
    assert np.abs(got3 - want3).max() <= tol


def test_noalloc_precompute_rejects_shapes_beyond_its_scratch():
    from paper_2510_18239_b200 import binding as Bd
    ell, d = 128, 256                               # 32768 link elements > 16384
    links = torch.zeros((ell, d), dtype=torch.bfloat16, device="cuda")
    cand = torch.zeros((4, d), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros((4, ell), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(Bd.LimeError) as e:
        Bd.lime_precompute_candidate_links_noalloc(Bd.LIME_BF16, d, ell, 0.0, links, None, None, cand, out)
    assert e.value.status == 7 and "LIME_NOALLOC_MAX_LINK_ELEMS" in str(e.value)
    assert torch.count_nonzero(out).item() == 0     # nothing was launched

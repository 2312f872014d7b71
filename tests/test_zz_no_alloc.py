"""tw_joiner_expand_noalloc: the handle-free, allocation-free packaging of the joiner + expansion
stage, meant for processes whose device memory is owned by another allocator.  It must give what
tw_joiner_expand gives, and what the oracle's joiner -> softmax -> Eq. 3-7 chain gives, call after call,
although all calls share one fixed scratch array that still holds the previous call's data.  The file
name sorts last so that a run that stops at the first failure has run every other test before it."""
import numpy as np
import pytest

import tw_synth
from oracle import rnnt_model as rm
from oracle import segment_math as sm
from helpers import oracle_model

pytestmark = pytest.mark.gpu
STAGE_TOL = 1e-5


def _case(rng, cfg, S, G, R):
    enc = rng.standard_normal((G, S, cfg.D_enc)).astype(np.float32)
    pred = rng.standard_normal((R, cfg.P)).astype(np.float32)
    row_group = rng.integers(0, G, size=R).astype(np.int32)
    seg_len = rng.integers(1, S + 1, size=G).astype(np.int32)
    ld_old = (rng.standard_normal((R, S)) - 2).astype(np.float32)
    ld_old[0, 1:] = -np.inf
    return enc, pred, row_group, seg_len, ld_old


def _close(got, want, tol):
    got, want = np.asarray(got, np.float64), np.asarray(want, np.float64)
    assert np.array_equal(np.isneginf(got), np.isneginf(want))
    fin = np.isfinite(want)
    np.testing.assert_allclose(got[fin], want[fin], rtol=1.2e-7, atol=tol)


@pytest.mark.parametrize("act", ["tanh", "relu"])
def test_noalloc_entry_point_matches_handle_path_and_oracle_twice_in_a_row(act):
    import torch
    from paper_2302_14357_b200 import binding
    cfg = tw_synth.WorkloadConfig("na", 4, 16, (16, 16), 24, "stateless", 20, 0, 0, 40, 150, 2.0, 3, (5,), "f32", 17, act)
    S = 5
    m = tw_synth.make_model(cfg)
    om = oracle_model(m)
    dec = binding.TwDecoder(binding.weights_from_synth(m), N=3, S=S, max_batch=8, max_T=16, joiner_act=act)
    W_out = torch.from_numpy(m.W_out).cuda()
    b_out = torch.from_numpy(m.b_out).cuda()
    rng = np.random.default_rng(5)
    # second call is smaller than the first: the scratch still holds the first call's rows
    for G, R in ((4, 21), (2, 6)):
        enc, pred, row_group, seg_len, ld_old = _case(rng, cfg, S, G, R)
        E = dec.project_encoder(enc).reshape(G, S, cfg.J)
        Pp = torch.from_numpy((pred.astype(np.float64) @ om.W_p.T).astype(np.float32)).cuda()   # input marshalling only
        rg, sl, lo = [torch.from_numpy(x).cuda() for x in (row_group, seg_len, ld_old)]
        ref = dec.joiner_expand(E, Pp, rg, sl, lo)
        st, ldphi, ldnb, la = binding.joiner_expand_noalloc(W_out, b_out, S, 0, E, Pp, rg, sl, lo, joiner_act=act)
        torch.cuda.synchronize()
        assert st == 0
        got = [x.cpu().numpy() for x in (ldphi, ldnb, la)]
        for g, want in zip(got, ref):
            _close(g, want.cpu().numpy(), STAGE_TOL)
        for r in range(R):
            n = seg_len[row_group[r]]
            lj = rm.joiner_log_probs(om, enc[row_group[r], :n], pred[r:r + 1])
            d0 = ld_old[r:r + 1, :n].astype(np.float64)
            lBl = sm.blank_product(lj)
            ld = sm.nonblank_expansion_t(lj, lBl, d0)
            _close(got[1][r], sm.nonblank_expansion(ld)[0], STAGE_TOL)
            _close(got[0][r:r + 1], sm.blank_expansion(lBl, d0), STAGE_TOL)
            _close((got[2][r, :n, None].astype(np.float64) + lj[0])[:, 1:], ld[0, 1:, :].T, STAGE_TOL)
            assert np.all(np.isneginf(got[2][r, n:]))
    dec.close()


def test_noalloc_entry_point_rejects_oversize_requests():
    import torch
    from paper_2302_14357_b200 import binding
    V, J, S = 1024, 8, 64
    W_out = torch.zeros((V, J), device="cuda")
    b_out = torch.zeros((V,), device="cuda")
    R = binding.NOALLOC_MAX_ELEMS // (S * V) + 1            # one row too many for the fixed array
    E = torch.zeros((1, S, J), device="cuda")
    Pp = torch.zeros((R, J), device="cuda")
    rg = torch.zeros((R,), dtype=torch.int32, device="cuda")
    ld = torch.zeros((R, S), device="cuda")
    st, *_ = binding.joiner_expand_noalloc(W_out, b_out, S, 0, E, Pp, rg, None, ld)
    assert st == 4                                           # TW_ERR_LIMIT, nothing enqueued
    st, *_ = binding.joiner_expand_noalloc(W_out, b_out, S, V, E, Pp[:1], rg[:1], None, ld[:1])
    assert st == 1                                           # blank outside the vocabulary
    st, *_ = binding.joiner_expand_noalloc(W_out, b_out, S, 0, E, Pp[:1], rg[:1], None, ld[:1], joiner_act=7)
    assert st == 1                                           # no such nonlinearity

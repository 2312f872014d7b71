"""Stage parity, CUDA path (through the C ABI) against the fp64 oracle, fp32 mode: joiner + softmax,
Eq. 3-7, predictor step.  Tolerance 1e-5 on log-probabilities."""
import numpy as np
import pytest

import tw_synth
from oracle import rnnt_model as rm
from oracle import segment_math as sm
from helpers import oracle_model

pytestmark = pytest.mark.gpu
STAGE_TOL = 1e-5


def _decoder(cfg, S, N=None, max_batch=8, mode=0):
    from paper_2302_14357_b200.binding import TwDecoder, weights_from_synth
    m = tw_synth.make_model(cfg)
    dec = TwDecoder(weights_from_synth(m), N=N or cfg.N, S=S, mode=mode, max_batch=max_batch, max_T=cfg.T)
    return m, dec


def _small_cfg(pred="lstm", V=70, J=48, D=40, emb=24, hidden=36, layers=2, seed=3):
    return tw_synth.WorkloadConfig("small", 4, 30, (7, 30), D, pred, emb, layers if pred == "lstm" else 0,
                                   hidden if pred == "lstm" else 0, J, V, 2.0, 4, (3,), "f32", seed)


def _allclose_inf(a, b, tol):
    a, b = np.asarray(a, dtype=np.float64), np.asarray(b, dtype=np.float64)
    assert a.shape == b.shape
    inf_a, inf_b = np.isneginf(a), np.isneginf(b)
    assert np.array_equal(inf_a, inf_b)
    assert np.all(np.isfinite(a[~inf_a]))
    # outputs are float32: beyond the stage tolerance allow the rounding of the stored value itself
    np.testing.assert_allclose(a[~inf_a], b[~inf_a], rtol=1.2e-7, atol=tol)


@pytest.mark.parametrize("S,seg_lens", [(1, None), (3, None), (5, [5, 2, 4]), (17, [17, 1, 9])])
def test_joiner_segment_matches_oracle(S, seg_lens):
    cfg = _small_cfg()
    m, dec = _decoder(cfg, S)
    om = oracle_model(m)
    rng = np.random.default_rng(S)
    G = 3
    enc = rng.standard_normal((G, S, cfg.D_enc)).astype(np.float32)
    row_group = np.array([0, 0, 1, 2, 2, 2, 1], dtype=np.int32)
    R = len(row_group)
    pred = rng.standard_normal((R, cfg.P)).astype(np.float32)
    E = dec.project_encoder(enc).reshape(G, S, cfg.J)
    Pp = (pred.astype(np.float64) @ om.W_p.T).astype(np.float32)     # input marshalling only
    got = dec.joiner_segment(E, Pp, row_group, seg_lens).cpu().numpy()
    for r in range(R):
        g = row_group[r]
        sl = S if seg_lens is None else seg_lens[g]
        ref = rm.joiner_log_probs(om, enc[g, :sl], pred[r:r + 1])[0]
        np.testing.assert_allclose(got[r, :sl], ref, rtol=0, atol=STAGE_TOL)
        assert np.all(got[r, sl:, 0] == 0.0) and np.all(np.isneginf(got[r, sl:, 1:]))


def test_joiner_spans_tiles_and_ragged_tail_on_config_shapes():
    """A C1-shaped joiner (J=640, V=1024) with a row count that is not a tile multiple."""
    cfg = tw_synth.get_config("c1")
    m, dec = _decoder(cfg, 3, max_batch=16)
    om = oracle_model(m)
    rng = np.random.default_rng(0)
    G, S, R = 5, 3, 23
    enc = tw_synth.round_to_bf16(rng.standard_normal((G, S, cfg.D_enc)).astype(np.float32))
    row_group = rng.integers(0, G, size=R).astype(np.int32)
    pred = rng.standard_normal((R, cfg.P)).astype(np.float32) * 0.3
    E = dec.project_encoder(enc).reshape(G, S, cfg.J)
    Pp = (pred.astype(np.float64) @ om.W_p.T).astype(np.float32)
    got = dec.joiner_segment(E, Pp, row_group).cpu().numpy()
    for r in range(R):
        ref = rm.joiner_log_probs(om, enc[row_group[r]], pred[r:r + 1])[0]
        np.testing.assert_allclose(got[r], ref, rtol=0, atol=STAGE_TOL)


@pytest.mark.parametrize("S", [1, 2, 3, 10, 50])
def test_expand_matches_explicit_sums(S):
    cfg = _small_cfg(V=130)
    m, dec = _decoder(cfg, S)
    rng = np.random.default_rng(100 + S)
    R, V = 6, cfg.V
    logJ = rm.log_softmax(rng.standard_normal((R, S, V)) * 2.0)
    ld_old = rng.standard_normal((R, S)) * 2 - 3
    ld_old[0, 1:] = -np.inf                       # segment start: all mass on frame 1
    if S > 1:
        ld_old[1, 0] = -np.inf
    seg = np.full(R, S, dtype=np.int32)
    if S > 2:
        seg[2], seg[3] = 1, S - 1                 # ragged last segments
    logJ32, ld32 = logJ.astype(np.float32), ld_old.astype(np.float32)
    ldphi, ldnb, la = [x.cpu().numpy() for x in dec.expand(logJ32, ld32, seg)]
    for r in range(R):
        sl = seg[r]
        lj = logJ32[r:r + 1, :sl].astype(np.float64)
        lo = ld32[r:r + 1, :sl].astype(np.float64)
        lBl = sm.blank_product(lj)
        ld = sm.nonblank_expansion_t(lj, lBl, lo)
        _allclose_inf(ldnb[r], sm.nonblank_expansion(ld)[0], STAGE_TOL)
        _allclose_inf(ldphi[r:r + 1], sm.blank_expansion(lBl, lo), STAGE_TOL)
        # la[t] + logJ[t, k] is log d(k, t) of Eq. 5
        d_gpu = la[r, :sl, None].astype(np.float64) + lj[0]
        _allclose_inf(d_gpu[:, 1:], ld[0, 1:, :].T, STAGE_TOL)
        assert np.all(np.isneginf(la[r, sl:]))


def test_expand_all_mass_missing_row():
    """A row whose d_old is all zero (log = -inf) yields log 0 everywhere, not NaN."""
    cfg = _small_cfg(V=40)
    m, dec = _decoder(cfg, 3)
    logJ = rm.log_softmax(np.random.default_rng(1).standard_normal((1, 3, 40))).astype(np.float32)
    ldphi, ldnb, la = [x.cpu().numpy() for x in dec.expand(logJ, np.full((1, 3), -np.inf, np.float32))]
    assert np.isneginf(ldphi).all() and np.isneginf(ldnb).all() and np.isneginf(la).all()


def test_joiner_expand_is_the_composition():
    cfg = _small_cfg()
    S = 4
    m, dec = _decoder(cfg, S)
    rng = np.random.default_rng(9)
    G, R = 2, 5
    E = rng.standard_normal((G, S, cfg.J)).astype(np.float32)
    Pp = rng.standard_normal((R, cfg.J)).astype(np.float32)
    row_group = np.array([0, 1, 1, 0, 1], np.int32)
    seg_len = np.array([4, 3], np.int32)
    ld_old = (rng.standard_normal((R, S)) - 2).astype(np.float32)
    logp = dec.joiner_segment(E, Pp, row_group, seg_len)
    a = dec.expand(logp, ld_old, seg_len[row_group])
    b = dec.joiner_expand(E, Pp, row_group, seg_len, ld_old)
    for x, y in zip(a, b):
        _allclose_inf(x.cpu().numpy(), y.cpu().numpy(), 1e-5)


@pytest.mark.parametrize("S,V", [(1, 70), (3, 1000), (10, 257), (50, 130)])
def test_joiner_expand_matches_oracle_chain(S, V):
    """The one-call stage against joiner -> softmax -> Eq. 3-7 of the oracle, ragged segments."""
    cfg = _small_cfg(V=V)
    m, dec = _decoder(cfg, S)
    om = oracle_model(m)
    rng = np.random.default_rng(S * 7 + V)
    G, R = 3, 6
    enc = rng.standard_normal((G, S, cfg.D_enc)).astype(np.float32)
    pred = rng.standard_normal((R, cfg.P)).astype(np.float32)
    row_group = np.array([0, 1, 2, 2, 1, 0], np.int32)
    seg_len = np.array([S, max(1, S // 2), max(1, S - 1)], np.int32)
    ld_old = (rng.standard_normal((R, S)) - 2).astype(np.float32)
    ld_old[0, 1:] = -np.inf
    E = dec.project_encoder(enc).reshape(G, S, cfg.J)
    Pp = (pred.astype(np.float64) @ om.W_p.T).astype(np.float32)
    ldphi, ldnb, la = [x.cpu().numpy() for x in dec.joiner_expand(E, Pp, row_group, seg_len, ld_old)]
    for r in range(R):
        sl = seg_len[row_group[r]]
        lj = rm.joiner_log_probs(om, enc[row_group[r], :sl], pred[r:r + 1])
        lo = ld_old[r:r + 1, :sl].astype(np.float64)
        lBl = sm.blank_product(lj)
        ld = sm.nonblank_expansion_t(lj, lBl, lo)
        _allclose_inf(ldnb[r], sm.nonblank_expansion(ld)[0], 2 * STAGE_TOL)
        _allclose_inf(ldphi[r:r + 1], sm.blank_expansion(lBl, lo), 2 * STAGE_TOL)


@pytest.mark.parametrize("pred,layers", [("stateless", 0), ("lstm", 1), ("lstm", 2)])
def test_predictor_step_matches_oracle(pred, layers):
    cfg = _small_cfg(pred=pred, layers=layers)
    m, dec = _decoder(cfg, 2)
    om = oracle_model(m)
    rng = np.random.default_rng(4)
    R = 7
    tokens = rng.integers(0, cfg.V, size=R).astype(np.int32)
    if pred == "stateless":
        _, Pp = dec.predictor_step(tokens)
        ref = om.emb[tokens] @ om.W_p.T
        np.testing.assert_allclose(Pp.cpu().numpy(), ref, atol=STAGE_TOL)
        return
    Hd = cfg.lstm_hidden
    state = (rng.standard_normal((R, layers, 2, Hd)) * 0.5).astype(np.float32)
    out, Pp = dec.predictor_step(tokens, state)
    out, Pp = out.cpu().numpy(), Pp.cpu().numpy()
    for r in range(R):
        st = ([state[r, l, 0].astype(np.float64) for l in range(layers)], [state[r, l, 1].astype(np.float64) for l in range(layers)])
        (h, c), o = rm.lstm_step(om, st, int(tokens[r]))
        for l in range(layers):
            np.testing.assert_allclose(out[r, l, 0], h[l], atol=STAGE_TOL)
            np.testing.assert_allclose(out[r, l, 1], c[l], atol=STAGE_TOL)
        np.testing.assert_allclose(Pp[r], om.W_p @ o, atol=STAGE_TOL)


def test_argument_errors_are_reported_not_launched():
    from paper_2302_14357_b200.binding import TwDecoder, TwError, weights_from_synth
    cfg = _small_cfg()
    m = tw_synth.make_model(cfg)
    w = weights_from_synth(m)
    for bad in (dict(N=0), dict(N=17), dict(S=0), dict(S=65), dict(N=cfg.V)):
        kw = dict(N=2, S=2, max_batch=2, max_T=10)
        kw.update(bad)
        with pytest.raises(TwError) as e:
            TwDecoder(w, **kw)
        assert e.value.status == 1
    dec = TwDecoder(w, N=2, S=2, max_batch=2, max_T=10)
    with pytest.raises(TwError):
        dec.decode(np.zeros((3, 10, cfg.D_enc), np.float32), np.array([1, 2, 3], np.int32))   # B > max_batch
    with pytest.raises(TwError):
        dec.decode(np.zeros((1, 11, cfg.D_enc), np.float32), np.array([1], np.int32))         # T > max_T

"""Blank thresholding on a factorised (HAT) joiner output (Sec. 2 and Sec. 5 name it; the rule is the one the
oracle states): a (hypothesis, frame) pair whose blank probability exceeds the threshold keeps its blank arc only.
fp32 mode: stage values within 1e-5 and identical N-best; bf16 mode: stage values within 2e-2, top-1 agreement."""
import numpy as np
import pytest

import tw_synth
from oracle import rnnt_model as rm
from oracle import segment_math as sm
from oracle import token_wise_search as tws
from helpers import check_against_oracle, nbest_from_arrays, oracle_model

pytestmark = pytest.mark.gpu
TOP1_GAP = 0.05


def _cfg(pred="lstm", V=24, J=16, D=12, emb=10, hidden=14, layers=1, seed=5, batch=6, T=23, bias=0.5, dtype="f32", N=3):
    return tw_synth.WorkloadConfig("hat", batch, T, (0, T), D, pred, emb, layers if pred == "lstm" else 0,
                                   hidden if pred == "lstm" else 0, J, V, bias, N, (2,), dtype, seed, "tanh", "hat")


def _decoder(cfg, S, mode=0, max_batch=None, N=None, max_T=None):
    from paper_2302_14357_b200.binding import TwDecoder, weights_from_synth
    m = tw_synth.make_model(cfg)
    return m, TwDecoder(weights_from_synth(m), N=N or cfg.N, S=S, mode=mode, max_batch=max_batch or cfg.batch, max_T=max_T or cfg.T)


def test_threshold_needs_a_factorised_model():
    cfg = _cfg().with_(joiner_norm="softmax")
    m, dec = _decoder(cfg, 2)
    assert dec.set_blank_threshold(0.5) == 5           # TW_ERR_STATE
    dec.close()
    m, dec = _decoder(_cfg(), 2)
    assert dec.set_blank_threshold(1.5) == 1 and dec.set_blank_threshold(-0.1) == 1
    assert dec.set_blank_threshold(0.7) == 0
    dec.close()


@pytest.mark.parametrize("tau", [1.0, 0.6, 0.0])
def test_joiner_segment_factorised_fp32(tau):
    cfg = _cfg(V=70, J=48, D=40)
    S, G, R = 4, 3, 9
    m, dec = _decoder(cfg, S, max_batch=4)
    assert dec.set_blank_threshold(tau) == 0
    om = oracle_model(m)
    rng = np.random.default_rng(int(tau * 10))
    enc = rng.standard_normal((G, S, cfg.D_enc)).astype(np.float32)
    row_group = rng.integers(0, G, size=R).astype(np.int32)
    seg_len = np.array([4, 2, 3], np.int32)
    pred = rng.standard_normal((R, cfg.P)).astype(np.float32)
    E = dec.project_encoder(enc).reshape(G, S, cfg.J)
    Pp = (pred.astype(np.float64) @ om.W_p.T).astype(np.float32)
    got = dec.joiner_segment(E, Pp, row_group, seg_len).cpu().numpy()
    skipped = 0
    for r in range(R):
        sl = seg_len[row_group[r]]
        full = rm.joiner_log_probs(om, enc[row_group[r], :sl], pred[r:r + 1])[0]
        np.testing.assert_allclose(np.exp(full).sum(axis=-1), 1.0, atol=1e-12)
        ref, skip = rm.apply_blank_threshold(full, tau, 0)
        for t in range(sl):
            with np.errstate(divide="ignore"):
                if abs(full[t, 0] - np.log(tau)) < 1e-5:
                    continue                           # a decision this close may fall either way in float32
            assert np.array_equal(np.isneginf(got[r, t]), np.isneginf(ref[t]))
            fin = np.isfinite(ref[t])
            np.testing.assert_allclose(got[r, t][fin], ref[t][fin], rtol=0, atol=1e-5)
        skipped += int(skip.sum())
    assert (skipped > 0) == (tau < 1.0)
    dec.close()


@pytest.mark.parametrize("pred,layers", [("stateless", 0), ("lstm", 2)])
@pytest.mark.parametrize("S,tau", [(1, 0.7), (3, 1.0), (3, 0.75), (4, 0.5), (3, 0.0)])
def test_decode_fp32_with_blank_threshold_matches_oracle(pred, layers, S, tau):
    cfg = _cfg(pred, layers=layers)
    m, dec = _decoder(cfg, S)
    assert dec.set_blank_threshold(tau) == 0
    enc, _ = tw_synth.make_encoder_batch(cfg)
    lens = np.array([0, 1, 23, 5, 17, 4], np.int32)
    tokens, olens, scores, status = [x.cpu().numpy() for x in dec.decode(enc, lens)[:4]]
    st = dec.stats()
    om = oracle_model(m)
    skipped = frame_rows = 0
    exact = True
    for b in range(cfg.batch):
        got = nbest_from_arrays(tokens, olens, scores, b)
        ok, why, ost = check_against_oracle(om, enc[b, :lens[b]], cfg.N, S, 4 * S + 16, got, blank_threshold=tau)
        assert ok, "utterance %d: %s" % (b, why)
        exact &= why == "exact"
        skipped += ost.skipped
        frame_rows += ost.frame_rows
    if exact:
        assert st["frame_rows_skipped"] == skipped and st["joiner_frame_rows"] == frame_rows
    assert (st["frame_rows_skipped"] > 0) == (tau < 1.0)
    if tau == 0.0:
        assert np.all(olens[lens > 0, 0] == 0) and st["frame_rows_skipped"] == st["joiner_frame_rows"]
    dec.close()


def _stage_case(cfg, m, dec, S, R, G, seed):
    om = oracle_model(m)
    rng = np.random.default_rng(seed)
    enc = tw_synth.round_to_bf16(rng.standard_normal((G, S, cfg.D_enc)).astype(np.float32))
    row_group = np.sort(rng.integers(0, G, size=R)).astype(np.int32)
    seg_len = rng.integers(1, S + 1, size=G).astype(np.int32)
    seg_len[rng.random(G) < 0.7] = S
    pred = (rng.standard_normal((R, cfg.P)) * 0.5).astype(np.float32)
    ld_old = (rng.standard_normal((R, S)) * 1.5 - 2).astype(np.float32)
    ld_old[::4, 1:] = -np.inf
    E = dec.project_encoder(enc).reshape(G, S, cfg.J)
    Pp = (pred.astype(np.float64) @ om.W_p.T).astype(np.float32)
    got = [x.cpu().numpy().astype(np.float64) for x in dec.joiner_expand(E, Pp, row_group, seg_len, ld_old)]
    return om, enc, pred, ld_old, row_group, seg_len, got


@pytest.mark.parametrize("V,J,S,R,tau,fused", [(512, 128, 3, 700, 0.8, True), (1024, 640, 3, 1700, 0.8, True), (1024, 640, 5, 900, 1.0, True),
                                               (512, 128, 10, 200, 0.7, True), (500, 128, 3, 300, 0.8, True), (512, 128, 3, 300, 0.8, False)])
def test_joiner_expand_bf16_with_blank_threshold(V, J, S, R, tau, fused):
    """The fused kernel (several tiles per cluster at the larger sizes, a padded vocabulary at V = 500) and the staged
    kernels on a factorised model: delta_phi, delta_nb and the occupancy of every row against the oracle.  Rows with a
    frame whose blank log-probability is within 4e-3 of the threshold may fall either way and are left out
    of the element-wise comparison (they are few)."""
    cfg = _cfg(V=V, J=J, D=64, emb=64, hidden=64, layers=1, bias=1.5, dtype="bf16", N=16)
    m, dec = _decoder(cfg, S, mode=1, max_batch=(R + 15) // 16, N=16, max_T=max(8, S * 17))
    assert dec.set_fused(fused) or not fused
    assert dec.set_blank_threshold(tau) == 0
    G = (R + 15) // 16
    om, enc, pred, ld_old, row_group, seg_len, (phi, nb, la) = _stage_case(cfg, m, dec, S, R, G, V + S)
    dec.close()
    checked = skipped_pairs = 0
    for g in np.unique(row_group):
        rows = np.nonzero(row_group == g)[0]
        sl = int(seg_len[g])
        full = rm.joiner_log_probs(om, enc[g, :sl], pred[rows])
        lj, skip = rm.apply_blank_threshold(full, tau, 0)
        lo = ld_old[rows, :sl].astype(np.float64)
        lBl = sm.blank_product(lj)
        ld = sm.nonblank_expansion_t(lj, lBl, lo)
        rnb = sm.nonblank_expansion(ld)
        rphi = sm.blank_expansion(lBl, lo)
        with np.errstate(divide="ignore"):
            close = (np.abs(full[..., 0] - np.log(tau)) < 4e-3).any(axis=1)   # log p(blank) moves by about a fifth of the logit's bf16 error
        for i, r in enumerate(rows):
            if close[i]:
                continue
            checked += 1
            skipped_pairs += int(skip[i].sum())
            if np.isfinite(rphi[i]):
                assert abs(phi[r] - rphi[i]) < 2e-2
            else:
                assert np.isneginf(phi[r])
            inf_ref = np.isneginf(rnb[i])
            assert np.array_equal(np.isneginf(nb[r]), inf_ref), (r, "log 0 pattern of delta_nb")
            assert np.abs(nb[r][~inf_ref] - rnb[i][~inf_ref]).max(initial=0.0) < 2e-2
    assert checked >= 0.8 * R
    assert (skipped_pairs > 0) == (tau < 1.0)


@pytest.mark.parametrize("fused", [True, False])
@pytest.mark.parametrize("tau", [1.0, 0.85])
def test_decode_bf16_with_blank_threshold_top1(fused, tau):
    cfg = tw_synth.get_config("h1")
    batch, T, S = 6, 60, 3
    from paper_2302_14357_b200.binding import MODE_BF16, TwDecoder, weights_from_synth
    m = tw_synth.make_model(cfg)
    enc, lens = tw_synth.make_encoder_batch(cfg, batch)
    enc, lens = np.ascontiguousarray(enc[:, :T]), np.minimum(lens, T)
    dec = TwDecoder(weights_from_synth(m), N=cfg.N, S=S, mode=MODE_BF16, max_batch=batch, max_T=T)
    assert dec.set_fused(fused) and dec.set_blank_threshold(tau) == 0
    tokens, olens, scores, status = [x.cpu().numpy() for x in dec.decode(enc, lens)[:4]]
    st = dec.stats()
    om = oracle_model(m)
    agree, gap, skipped, frame_rows = 0, 0.0, 0, 0
    for b in range(batch):
        ref, ost = tws.token_wise_beam_search(om, enc[b, :lens[b]], cfg.N, S, max_iters=4 * S + 16, blank_threshold=tau)
        got = nbest_from_arrays(tokens, olens, scores, b)
        skipped += ost.skipped
        frame_rows += ost.frame_rows
        if got[0][0] == ref[0][0]:
            agree += 1
            gap = max(gap, abs(got[0][1] - ref[0][1]))
    print("h1 tau=%.2f fused=%s: top-1 %d/%d, gap %.3g, skipped %d of %d pairs (oracle %d of %d)"
          % (tau, fused, agree, batch, gap, st["frame_rows_skipped"], st["joiner_frame_rows"], skipped, frame_rows))
    assert agree >= batch - 1 and gap < TOP1_GAP
    assert np.all(status == 0)
    if tau < 1.0:
        assert st["frame_rows_skipped"] > 0.2 * st["joiner_frame_rows"]          # the workload's blank head makes skipping common
        assert abs(st["frame_rows_skipped"] - skipped) <= 0.1 * skipped + 5
    else:
        assert st["frame_rows_skipped"] == 0
    dec.close()

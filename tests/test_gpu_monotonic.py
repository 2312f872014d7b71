"""Monotonic RNN-T variant (tw_set_monotonic: every output consumes a frame) against the oracle's monotonic
Algorithm 1: fp32 mode gives the identical N-best (scores within 1e-4, near-tie protocol), the bf16 path the
same top-1, streaming the same result as the offline decode."""
import numpy as np
import pytest

import tw_synth
from oracle import token_wise_search as tws
from helpers import check_against_oracle, nbest_from_arrays, oracle_model

pytestmark = pytest.mark.gpu


def _tiny(pred, layers=1, V=20, seed=5, batch=6, T=23, blank_bias=1.5, dtype="f32", J=16, D=12, emb=10, hidden=14):
    return tw_synth.WorkloadConfig("t", batch, T, (0, T), D, pred, emb, layers if pred == "lstm" else 0,
                                   hidden if pred == "lstm" else 0, J, V, blank_bias, 3, (2,), dtype, seed)


def _decode(cfg, S, N, mode=0, lengths=None, monotonic=True, fused=None):
    from paper_2302_14357_b200.binding import TwDecoder, weights_from_synth
    m = tw_synth.make_model(cfg)
    enc, lens = tw_synth.make_encoder_batch(cfg)
    if lengths is not None:
        lens = np.asarray(lengths, dtype=np.int32)
    dec = TwDecoder(weights_from_synth(m), N=N, S=S, mode=mode, max_batch=enc.shape[0], max_T=enc.shape[1])
    dec.set_monotonic(monotonic)
    if fused is not None:
        assert dec.set_fused(fused)
    out = [x.cpu().numpy() for x in dec.decode(enc, lens)[:4]]
    stats = dec.stats()
    return m, enc, lens, out, stats, dec


@pytest.mark.parametrize("pred,layers", [("stateless", 0), ("lstm", 2)])
@pytest.mark.parametrize("S", [1, 2, 4, 30])
def test_monotonic_decode_equals_oracle(pred, layers, S):
    cfg = _tiny(pred, layers)
    N = 3
    m, enc, lens, (tokens, olens, scores, status), stats, dec = _decode(cfg, S, N, lengths=[0, 1, 23, 5, 17, 4])
    om = oracle_model(m)
    calls = joins = 0
    exact = True
    for b in range(enc.shape[0]):
        got = nbest_from_arrays(tokens, olens, scores, b)
        ok, why, st = check_against_oracle(om, enc[b, :lens[b]], N, S, 4 * S + 16, got, monotonic=True)
        assert ok, "utterance %d (S=%d): %s" % (b, S, why)
        assert status[b] == 0 and not st.limit_hit
        assert all(len(t) <= lens[b] for t, _ in got)           # at most one token per frame
        exact &= why == "exact"
        calls += st.calls
        joins += st.joins
    if exact:
        assert stats["calls"] == calls and stats["joins"] == joins
    # switching the variant off again restores the standard search on the same handle
    dec.set_monotonic(False)
    t2, l2, s2, _ = [x.cpu().numpy() for x in dec.decode(enc, lens)[:4]]
    ok, why, _ = check_against_oracle(om, enc[2, :lens[2]], N, S, 4 * S + 16, nbest_from_arrays(t2, l2, s2, 2))
    assert ok, why
    dec.close()


def test_monotonic_is_a_different_search():
    """Same handle, same input: the variant changes the scores (a different lattice), and no monotonic
    hypothesis is longer than its utterance."""
    cfg = _tiny("lstm", 1)
    m, enc, lens, (tokens, olens, scores, status), _, dec = _decode(cfg, 3, 3)
    assert np.all(olens <= lens[:, None])
    dec.set_monotonic(False)
    s2 = dec.decode(enc, lens)[2].cpu().numpy()
    assert np.sum(np.abs(scores[:, 0] - s2[:, 0]) > 1e-3) >= 3
    dec.close()


@pytest.mark.parametrize("S,fused", [(3, True), (3, False), (10, True)])
def test_monotonic_bf16_top1(S, fused):
    cfg = _tiny("lstm", 2, V=512, J=128, D=64, emb=64, hidden=64, dtype="bf16", batch=6, T=40, blank_bias=3.0, seed=3)
    N = 4
    m, enc, lens, (tokens, olens, scores, status), stats, dec = _decode(cfg, S, N, mode=1, fused=fused)
    om = oracle_model(m)
    same = 0
    for b in range(enc.shape[0]):
        ref, _ = tws.token_wise_beam_search(om, enc[b, :lens[b]].astype(np.float64), N, S, max_iters=4 * S + 16, monotonic=True)
        got = nbest_from_arrays(tokens, olens, scores, b)
        same += int(got[0][0] == ref[0][0])
        if got[0][0] == ref[0][0]:
            assert abs(got[0][1] - ref[0][1]) < 0.05
    assert same >= enc.shape[0] - 1
    assert np.all(status == 0)
    dec.close()


@pytest.mark.parametrize("mode", [0, 1])
def test_monotonic_streaming_equals_offline(mode):
    from paper_2302_14357_b200.binding import TwError
    cfg = _tiny("lstm", 1, V=256, J=64, D=64, emb=32, hidden=32, dtype="bf16" if mode else "f32", batch=4, T=24)
    m, enc, lens, ref, _, dec = _decode(cfg, 3, 3, mode=mode)
    B = enc.shape[0]
    dec.stream_open(B)
    with pytest.raises(TwError):
        dec.set_monotonic(False)                               # not while a session is open
    t = 0
    for n in (5, 1, 11, 7):
        dec.stream_push(np.ascontiguousarray(enc[:, t:t + n]), np.clip(lens - t, 0, n).astype(np.int32))
        t += n
    got = [x.cpu().numpy() for x in dec.stream_close()[:4]]
    for x, y in zip(got, ref):
        np.testing.assert_array_equal(x, y)
    dec.close()

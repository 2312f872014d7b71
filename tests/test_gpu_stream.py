"""Streaming entry points: frames pushed in chunks of arbitrary sizes must give, after tw_stream_close,
exactly what tw_decode gives on the whole utterances (Sec. 3.2: the chunking of the encoder output need
not match the decoding segment size), and sensible N-best lists in between."""
import numpy as np
import pytest

import tw_synth
from helpers import check_against_oracle, nbest_from_arrays, oracle_model

pytestmark = pytest.mark.gpu


def _cfg(pred, batch=5, T=29):
    return tw_synth.WorkloadConfig("s", batch, T, (3, T), 16, pred, 16, 2 if pred == "lstm" else 0,
                                   24 if pred == "lstm" else 0, 32, 256, 2.0, 3, (3,), "bf16", 21)


@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("pred,S,chunks", [("lstm", 3, (4, 1, 7, 2, 9, 6)), ("stateless", 4, (10, 10, 9)), ("lstm", 1, (29,)),
                                           ("lstm", 5, (2, 2, 2, 2, 2, 2, 2, 2, 2, 2, 2, 2, 2, 2, 1))])
def test_streamed_chunks_equal_offline_decode(mode, pred, S, chunks):
    from paper_2302_14357_b200.binding import TwDecoder, weights_from_synth
    cfg = _cfg(pred)
    m = tw_synth.make_model(cfg)
    enc, lens = tw_synth.make_encoder_batch(cfg)
    lens[1] = 0
    B, T = enc.shape[0], enc.shape[1]
    assert sum(chunks) == T
    dec = TwDecoder(weights_from_synth(m), N=cfg.N, S=S, mode=mode, max_batch=B, max_T=T)
    ref = [x.cpu().numpy() for x in dec.decode(enc, lens)[:4]]
    ref_stats = dec.stats()

    dec.stream_open(B)
    t = 0
    for n in chunks:
        chunk = np.ascontiguousarray(enc[:, t:t + n])
        chunk_lens = np.clip(lens - t, 0, n).astype(np.int32)      # utterances end at their own lengths
        dec.stream_push(chunk, chunk_lens)
        t += n
        mid = [x.cpu().numpy() for x in dec.stream_nbest()]
        assert np.all(mid[1][:, 0] >= 0)
        with np.errstate(invalid="ignore"):
            assert not np.any(np.diff(mid[2], axis=1) > 0)      # best first (unused slots hold -inf)
    out = dec.stream_close()
    got = [x.cpu().numpy() for x in out[:4]]
    for x, y in zip(got, ref):
        np.testing.assert_array_equal(x, y)
    st = dec.stats()
    for key in ("frames", "calls", "joins"):
        assert st[key] == ref_stats[key], key
    # and the offline result itself is the oracle's (fp32 mode)
    if mode == 0:
        om = oracle_model(m)
        for b in (0, 2):
            ok, why, _ = check_against_oracle(om, enc[b, :lens[b]], cfg.N, S, 4 * S + 16, nbest_from_arrays(*got[:3], b))
            assert ok, why
    dec.close()


def test_stream_calls_without_session_and_overflow():
    from paper_2302_14357_b200.binding import TwDecoder, TwError, weights_from_synth
    cfg = _cfg("stateless", batch=2, T=8)
    m = tw_synth.make_model(cfg)
    enc, _ = tw_synth.make_encoder_batch(cfg)
    dec = TwDecoder(weights_from_synth(m), N=2, S=2, max_batch=2, max_T=8)
    with pytest.raises(TwError) as e:
        dec.stream_push(enc[:, :4], np.array([4, 4], np.int32))
    assert e.value.status == 5                                  # TW_ERR_STATE: no open session
    dec.stream_open(2)
    dec.stream_push(enc[:, :6], np.array([6, 6], np.int32))
    dec.stream_push(enc[:, :6], np.array([6, 1], np.int32))      # utterance 0 would exceed max_T = 8
    tokens, lens, scores, status, rc = dec.stream_close()
    assert status.cpu().numpy().tolist() == [4, 0] and rc == 4   # TW_ERR_LIMIT for the clipped utterance
    dec.close()

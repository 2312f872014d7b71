"""End-to-end parity of tw_decode (fp32 mode) with the oracle's Algorithm 1: identical N-best token
sequences, log-scores within 1e-4, same Calls/Frame and Joins/Frame counters."""
import numpy as np
import pytest

import tw_synth
from helpers import SCORE_TOL, check_against_oracle, nbest_from_arrays, oracle_model

pytestmark = pytest.mark.gpu


def _run(cfg, S, N=None, batch=None, T=None, lengths=None, max_iters=0, mode=0, check=None, mutate=None):
    from paper_2302_14357_b200.binding import TwDecoder, weights_from_synth
    N = N or cfg.N
    m = tw_synth.make_model(cfg)
    if mutate is not None:
        mutate(m)
    enc, lens = tw_synth.make_encoder_batch(cfg, batch)
    if T is not None:
        enc = np.ascontiguousarray(enc[:, :T])
        lens = np.minimum(lens, T)
    if lengths is not None:
        lens = np.asarray(lengths, dtype=np.int32)
    B = enc.shape[0]
    dec = TwDecoder(weights_from_synth(m), N=N, S=S, mode=mode, max_batch=B, max_T=enc.shape[1], max_iters_per_segment=max_iters)
    tokens, olens, scores, status, rc = dec.decode(enc, lens)
    tokens, olens, scores, status = [x.cpu().numpy() for x in (tokens, olens, scores, status)]
    stats = dec.stats()
    om = oracle_model(m)
    I_max = max_iters or 4 * S + 16
    calls = joins = 0
    how = []
    for b in (range(B) if check is None else check):
        got = nbest_from_arrays(tokens, olens, scores, b)
        ok, why, st = check_against_oracle(om, enc[b, :lens[b]], N, S, I_max, got)
        assert ok, "utterance %d (S=%d): %s" % (b, S, why)
        assert status[b] == (4 if st.limit_hit else 0)
        how.append(why)
        calls += st.calls
        joins += st.joins
    if check is None:
        assert stats["frames"] == int(lens.sum())
        if all(h == "exact" for h in how):
            assert stats["calls"] == calls and stats["joins"] == joins
    assert stats["kernel_launches"] > 0
    dec.close()
    return stats, how


@pytest.mark.parametrize("S", [1, 2, 3, 7, 40, 64])
def test_config0_all_segment_sizes(S):
    _run(tw_synth.get_config("c0"), S)


@pytest.mark.parametrize("N", [1, 2, 5, 16])
def test_config0_beam_sizes(N):
    _run(tw_synth.get_config("c0"), 3, N=N)


def _tiny(pred, layers=1, V=20, seed=5, batch=6, T=23, lo=0):
    return tw_synth.WorkloadConfig("t", batch, T, (lo, T), 12, pred, 10, layers if pred == "lstm" else 0,
                                   14 if pred == "lstm" else 0, 16, V, 1.5, 3, (2,), "f32", seed)


@pytest.mark.parametrize("pred,layers", [("stateless", 0), ("lstm", 1), ("lstm", 3)])
@pytest.mark.parametrize("S", [1, 4])
def test_small_models_ragged_batch(pred, layers, S):
    """Variable lengths incl. empty and one-frame utterances; S does not divide most lengths."""
    cfg = _tiny(pred, layers)
    _run(cfg, S, lengths=[0, 1, 23, 5, 17, 4])


@pytest.mark.parametrize("pred,layers,what", [("lstm", 2, "state"), ("lstm", 1, "both"), ("lstm", 2, "out"), ("stateless", 0, "out")])
def test_learned_initial_predictor_state(pred, layers, what):
    """InitPredictor() as a caller-supplied quantity (Sec. 3.2): state and / or output of the empty prefix."""
    cfg = _tiny(pred, layers, seed=13)
    rng = np.random.default_rng(layers + len(what))

    def mutate(m):
        if what in ("state", "both"):
            m.pred_init_state = (rng.standard_normal((layers, 2, cfg.lstm_hidden)) * 0.7).astype(np.float32)
        if what in ("out", "both"):
            m.pred_init_out = (rng.standard_normal(cfg.P) * 0.7).astype(np.float32)
    _run(cfg, 3, lengths=[0, 1, 23, 5, 17, 4], mutate=mutate)
    _run(cfg, 1, lengths=[3, 23, 2, 9, 1, 11], mutate=mutate)


def test_bf16_weights_and_frames_at_the_boundary():
    """tw_model::dtype = TW_BF16: weights and encoder frames cross the boundary as bfloat16.  On a bf16-representable
    workload the decode is the float32-boundary decode bit for bit, in both arithmetic modes, from device frames,
    from host frames (tw_decode_host) and as a streaming session."""
    import torch
    from paper_2302_14357_b200.binding import TwDecoder, weights_from_synth
    cfg = tw_synth.WorkloadConfig("bd", 5, 50, (20, 50), 64, "lstm", 64, 2, 64, 128, 256, 3.0, 4, (3,), "bf16", 9)
    m = tw_synth.make_model(cfg)
    enc, lens = tw_synth.make_encoder_batch(cfg)
    for mode in (0, 1):
        a = TwDecoder(weights_from_synth(m), N=4, S=3, mode=mode, max_batch=5, max_T=50, dtype="f32")
        b = TwDecoder(weights_from_synth(m), N=4, S=3, mode=mode, max_batch=5, max_T=50, dtype="bf16")
        ref = [x.cpu().numpy() for x in a.decode(enc, lens)[:4]]
        got = [x.cpu().numpy() for x in b.decode(torch.from_numpy(enc).to(torch.bfloat16).cuda(), lens)[:4]]
        for x, y in zip(got, ref):
            np.testing.assert_array_equal(x, y)
        host = b.decode_host(torch.from_numpy(enc).to(torch.bfloat16).contiguous(), lens)[:4]
        for x, y in zip(host, ref):
            np.testing.assert_array_equal(x, y)
        b.stream_open(5)
        for t0 in range(0, 50, 20):
            chunk = enc[:, t0:t0 + 20]
            b.stream_push(chunk, np.clip(lens - t0, 0, chunk.shape[1]))
        out = b.stream_close()
        for x, y in zip(out[:4], ref):
            np.testing.assert_array_equal(x.cpu().numpy(), y)
        # the stage call takes frames of the handle's element type too
        E_a = a.project_encoder(enc[0]).cpu().numpy()
        E_b = b.project_encoder(torch.from_numpy(enc[0]).to(torch.bfloat16)).cpu().numpy()
        np.testing.assert_array_equal(E_a, E_b)
        a.close()
        b.close()


def test_iteration_cap_sets_limit_status():
    cfg = _tiny("stateless", V=12, seed=8).with_(blank_bias=-2.0)
    stats, _ = _run(cfg, 3, N=3, max_iters=2, lengths=[9, 9, 9, 9, 9, 9])
    assert stats["limit_hits"] > 0


def test_many_merges_small_vocab():
    """V=3: few distinct sequences, so AddAndMerge fires constantly."""
    cfg = _tiny("lstm", 1, V=3, seed=12).with_(blank_bias=0.0)
    _run(cfg, 3, N=2, lengths=[23, 11, 23, 8, 2, 23])


def test_uniform_joiner_exact_ties():
    """W_out = 0: every token of a row has the same score, so the selection runs on ties alone
    (smaller hypothesis index, then smaller token) and more tokens tie than the fast path holds."""
    def flat(m):
        m.W_out[:] = 0.0
        m.b_out[:] = 0.0
    cfg = _tiny("stateless", V=300, seed=3)
    _run(cfg, 3, N=4, lengths=[7, 3, 6, 1, 2, 5], mutate=flat, max_iters=3)


@pytest.mark.parametrize("S", [1, 3])
def test_relu_joiner_small_model(S):
    cfg = _tiny("lstm", 2, V=33, seed=14).with_(joiner_act="relu")
    _run(cfg, S, lengths=[23, 6, 23, 1, 12, 19])


def test_paper_shaped_relu_workload_subset():
    """ReLU joiner, 3-layer LSTM predictor, 501-token vocabulary (not a multiple of 4)."""
    _run(tw_synth.get_config("p1"), 3, batch=3, T=60)


@pytest.mark.parametrize("S", [1, 2, 3, 5])
def test_config1_subset(S):
    _run(tw_synth.get_config("c1"), S, batch=3, T=90)


@pytest.mark.parametrize("S", [3, 10, 50])
def test_config2_subset(S):
    _run(tw_synth.get_config("c2"), S, batch=2, T=100)


def test_config3_subset():
    _run(tw_synth.get_config("c3"), 3, batch=2, T=45)


def test_config4_shape_subset():
    _run(tw_synth.get_config("c4"), 10, batch=3, T=40, lengths=[40, 25, 33])


@pytest.mark.parametrize("mode", [0, 1])
def test_two_lanes_give_the_single_lane_result(mode):
    """A large batch decoded as two concurrent halves (the default from 256 utterances up) equals the
    batch decoded in one piece: utterances never interact."""
    from paper_2302_14357_b200.binding import TwDecoder, weights_from_synth
    cfg = tw_synth.WorkloadConfig("lanes", 300, 24, (0, 24), 64, "lstm", 64, 1, 64, 64, 256, 3.0, 3, (3,), "bf16", 9)
    m = tw_synth.make_model(cfg)
    enc, lens = tw_synth.make_encoder_batch(cfg)
    dec = TwDecoder(weights_from_synth(m), N=cfg.N, S=3, mode=mode, max_batch=300, max_T=24)
    a = [x.cpu().numpy() for x in dec.decode(enc, lens)[:4]]
    sa = dec.stats()
    dec.set_lanes(False)
    b = [x.cpu().numpy() for x in dec.decode(enc, lens)[:4]]
    sb = dec.stats()
    for x, y in zip(a, b):
        np.testing.assert_array_equal(x, y)
    for key in ("frames", "calls", "joins", "rows", "limit_hits"):
        assert sa[key] == sb[key], key
    # an odd batch, and one below the lane threshold
    dec.set_lanes(True)
    c = [x.cpu().numpy() for x in dec.decode(enc[:257], lens[:257])[:4]]
    d = [x.cpu().numpy() for x in dec.decode(enc[:5], lens[:5])[:4]]
    for x, y in zip(c, a):
        np.testing.assert_array_equal(x, y[:257])
    for x, y in zip(d, a):
        np.testing.assert_array_equal(x, y[:5])
    dec.close()


def test_decode_host_equals_device_decode():
    from paper_2302_14357_b200.binding import TwDecoder, weights_from_synth
    cfg = tw_synth.get_config("c0")
    m = tw_synth.make_model(cfg)
    enc, lens = tw_synth.make_encoder_batch(cfg)
    dec = TwDecoder(weights_from_synth(m), N=2, S=2, max_batch=1, max_T=cfg.T)
    a = [x.cpu().numpy() for x in dec.decode(enc, lens)[:4]]
    b = dec.decode_host(enc, lens)[:4]
    for x, y in zip(a, b):
        np.testing.assert_array_equal(x, y)
    # repeated decodes on one handle give the same answer (workspace is re-initialised)
    c = dec.decode_host(enc, lens)[:4]
    for x, y in zip(b, c):
        np.testing.assert_array_equal(x, y)


@pytest.mark.parametrize("mode", [0, 1])
def test_decode_host_chunked_upload_ragged_batch(mode):
    """tw_decode_host uploads in time chunks and decodes each as it arrives: same result as tw_decode on device
    buffers, for ragged lengths (empty, one frame, full), and also when a length is out of range (which takes the
    plain path and reports the utterance)."""
    from paper_2302_14357_b200.binding import TwDecoder, weights_from_synth
    cfg = tw_synth.WorkloadConfig("h", 6, 64, (0, 64), 64, "lstm", 32, 1, 32, 64, 256, 2.0, 3, (3,), "bf16" if mode else "f32", 11)
    m = tw_synth.make_model(cfg)
    enc, lens = tw_synth.make_encoder_batch(cfg)
    lens[:] = [64, 0, 1, 37, 50, 63]
    dec = TwDecoder(weights_from_synth(m), N=3, S=3, mode=mode, max_batch=6, max_T=64)
    a = [x.cpu().numpy() for x in dec.decode(enc, lens)[:4]]
    b = dec.decode_host(enc, lens)[:4]
    for x, y in zip(a, b):
        np.testing.assert_array_equal(x, y)
    bad = lens.copy()
    bad[3] = 99
    c = dec.decode_host(enc, bad)
    assert c[3][3] == 1 and c[3][0] == 0           # TW_ERR_ARG for that utterance only
    np.testing.assert_array_equal(c[0][0], a[0][0])
    dec.close()

"""Pins for the CPU oracle: closed forms, hand-worked values, invariants, a
library LSTM, the frame-wise standard search and brute-force alignment sums.
Everything here runs without a GPU."""
import itertools
import math
import os

import numpy as np
import pytest

import tw_synth
from oracle import exact_forward as ef
from oracle import rnnt_model as rm
from oracle import segment_math as sm
from oracle import standard_search as ss
from oracle import token_wise_search as tws

from helpers import oracle_model, tiny_case

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _read_golden(name):
    rows = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append([float(x) for x in line.split()])
    return rows


def _random_logJ(rng, H, S, V, scale=2.0):
    return rm.log_softmax(rng.standard_normal((H, S, V)) * scale)


# ---------------------------------------------------------------- model pieces
def test_joiner_closed_form_golden():
    """Sec. 3.1 joiner + softmax on the hand-worked example (non-square shapes
    so that a transposed operand cannot pass)."""
    expected = np.array([r[0] for r in _read_golden("joiner_closed_form.txt")])
    model = rm.RnntModel(W_e=[[math.atanh(0.5)], [0.0]], W_p=[[0.0], [math.atanh(0.25)]],
                         W_out=[[2, 0], [0, 4], [2, 4]], b_out=[0, 0, 0], emb=np.zeros((3, 1)))
    out = rm.joiner_log_probs(model, np.array([[1.0]]), np.array([[1.0]]))
    assert out.shape == (1, 1, 3)
    np.testing.assert_allclose(out[0, 0], expected, atol=1e-14)


def test_relu_joiner_closed_form_golden():
    """The ReLU joiner of the paper's models on a hand-worked example; the negative pre-activation must
    be clipped (tanh would give a different third decimal)."""
    expected = np.array([r[0] for r in _read_golden("joiner_relu_closed_form.txt")])
    model = rm.RnntModel(W_e=[[0.5], [0.2]], W_p=[[0.0], [-0.5]], W_out=[[2, 7], [0, 3], [4, 1]],
                         b_out=[0, 0, 0], emb=np.zeros((3, 1)), activation="relu")
    out = rm.joiner_log_probs(model, np.array([[1.0]]), np.array([[1.0]]))
    np.testing.assert_allclose(out[0, 0], expected, atol=1e-14)
    tanh_model = rm.RnntModel(W_e=[[0.5], [0.2]], W_p=[[0.0], [-0.5]], W_out=[[2, 7], [0, 3], [4, 1]],
                              b_out=[0, 0, 0], emb=np.zeros((3, 1)))
    assert np.abs(rm.joiner_log_probs(tanh_model, np.array([[1.0]]), np.array([[1.0]]))[0, 0] - expected).max() > 0.05


def test_relu_model_unpruned_search_is_exact():
    cfg, model, enc = tiny_case(V=4, T=4, pred="lstm", seed=31)
    model.activation = "relu"
    nbest, _ = tws.token_wise_beam_search(model, enc, N=400, S=3, max_len=2)
    for y, s in nbest:
        assert s == pytest.approx(ef.forward_log_prob(model, enc, y), abs=1e-11)


def test_joiner_bias_and_broadcast_layout():
    """Output is [hypothesis, frame, vocab]; bias shifts one token's logit."""
    rng = np.random.default_rng(0)
    D, P, J, V, S, H = 3, 5, 7, 4, 2, 3
    args = dict(W_e=rng.standard_normal((J, D)), W_p=rng.standard_normal((J, P)),
                W_out=rng.standard_normal((V, J)), emb=np.zeros((V, P)))
    seg, pred = rng.standard_normal((S, D)), rng.standard_normal((H, P))
    base = rm.joiner_log_probs(rm.RnntModel(b_out=np.zeros(V), **args), seg, pred)
    assert base.shape == (H, S, V)
    np.testing.assert_allclose(np.exp(base).sum(-1), 1.0, atol=1e-13)
    # each (h, t) entry only depends on pred[h] and seg[t]
    single = rm.joiner_log_probs(rm.RnntModel(b_out=np.zeros(V), **args), seg[1:2], pred[2:3])
    np.testing.assert_allclose(single[0, 0], base[2, 1], atol=1e-13)
    # bias b on token 0: unnormalised ratio p0/pk scales by exp(b)
    b = np.zeros(V); b[0] = 1.5
    shifted = rm.joiner_log_probs(rm.RnntModel(b_out=b, **args), seg, pred)
    np.testing.assert_allclose((shifted[..., 0] - shifted[..., 1]) - (base[..., 0] - base[..., 1]), 1.5, atol=1e-12)


@pytest.mark.parametrize("layers", [1, 2])
def test_lstm_predictor_matches_library_lstm(layers):
    """The LSTM predictor against torch.nn.LSTM (fp64, CPU): same gate order
    (input, forget, cell, output), one bias per layer."""
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(3)
    V, E, Hd = 6, 5, 4
    W_ih = [rng.standard_normal((4 * Hd, E if l == 0 else Hd)) for l in range(layers)]
    W_hh = [rng.standard_normal((4 * Hd, Hd)) for l in range(layers)]
    b = [rng.standard_normal(4 * Hd) for l in range(layers)]
    emb = rng.standard_normal((V, E))
    model = rm.RnntModel(W_e=np.zeros((2, 3)), W_p=np.zeros((2, Hd)), W_out=np.zeros((V, 2)),
                         b_out=np.zeros(V), emb=emb, lstm_W_ih=W_ih, lstm_W_hh=W_hh, lstm_b=b)
    lib = torch.nn.LSTM(E, Hd, num_layers=layers).double()
    with torch.no_grad():
        for l in range(layers):
            getattr(lib, f"weight_ih_l{l}").copy_(torch.from_numpy(W_ih[l]))
            getattr(lib, f"weight_hh_l{l}").copy_(torch.from_numpy(W_hh[l]))
            getattr(lib, f"bias_ih_l{l}").copy_(torch.from_numpy(b[l]))
            getattr(lib, f"bias_hh_l{l}").zero_()
    tokens = [0, 3, 1, 5, 5]   # blank first: InitPredictor feeds the blank token from a zero state
    with torch.no_grad():
        out, _ = lib(torch.from_numpy(emb[tokens]).unsqueeze(1))
    state, o = rm.predictor_init(model)
    np.testing.assert_allclose(o, out[0, 0].numpy(), atol=1e-12)
    for i, k in enumerate(tokens[1:], start=1):
        state, o = rm.predictor_step(model, state, k)
        np.testing.assert_allclose(o, out[i, 0].numpy(), atol=1e-12)
    _, o2 = rm.predictor_for_tokens(model, tokens[1:])
    np.testing.assert_allclose(o2, o, atol=0)


@pytest.mark.parametrize("layers", [1, 3])
def test_lstm_step_rows_matches_library_lstm_cell_batch(layers):
    """The batched predictor step against torch.nn.LSTM run on a batch with given (h0, c0) (fp64, CPU), and
    against the one-row step: a transposed weight, a swapped gate or a mixed-up row would fail."""
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(11)
    V, E, Hd, R = 7, 5, 6, 9
    W_ih = [rng.standard_normal((4 * Hd, E if l == 0 else Hd)) for l in range(layers)]
    W_hh = [rng.standard_normal((4 * Hd, Hd)) for l in range(layers)]
    b = [rng.standard_normal(4 * Hd) for l in range(layers)]
    emb = rng.standard_normal((V, E))
    model = rm.RnntModel(W_e=np.zeros((2, 3)), W_p=np.zeros((2, Hd)), W_out=np.zeros((V, 2)),
                         b_out=np.zeros(V), emb=emb, lstm_W_ih=W_ih, lstm_W_hh=W_hh, lstm_b=b)
    h0, c0 = rng.standard_normal((R, layers, Hd)), rng.standard_normal((R, layers, Hd))
    tokens = rng.integers(0, V, size=R)
    h1, c1, out = rm.lstm_step_rows(model, h0, c0, tokens)
    lib = torch.nn.LSTM(E, Hd, num_layers=layers).double()
    with torch.no_grad():
        for l in range(layers):
            getattr(lib, f"weight_ih_l{l}").copy_(torch.from_numpy(W_ih[l]))
            getattr(lib, f"weight_hh_l{l}").copy_(torch.from_numpy(W_hh[l]))
            getattr(lib, f"bias_ih_l{l}").copy_(torch.from_numpy(b[l]))
            getattr(lib, f"bias_hh_l{l}").zero_()
        o_lib, (h_lib, c_lib) = lib(torch.from_numpy(emb[tokens]).unsqueeze(0),
                                    (torch.from_numpy(h0.transpose(1, 0, 2).copy()), torch.from_numpy(c0.transpose(1, 0, 2).copy())))
    np.testing.assert_allclose(out, o_lib[0].numpy(), atol=1e-12)
    np.testing.assert_allclose(h1, h_lib.numpy().transpose(1, 0, 2), atol=1e-12)
    np.testing.assert_allclose(c1, c_lib.numpy().transpose(1, 0, 2), atol=1e-12)
    for r in range(R):
        st = ([h0[r, l] for l in range(layers)], [c0[r, l] for l in range(layers)])
        (h, c), o = rm.lstm_step(model, st, int(tokens[r]))
        np.testing.assert_allclose(out[r], o, atol=1e-12)
        for l in range(layers):
            np.testing.assert_allclose(h1[r, l], h[l], atol=1e-12)
            np.testing.assert_allclose(c1[r, l], c[l], atol=1e-12)


def test_learned_initial_predictor_state_lstm():
    """InitPredictor() with a given state (Sec. 3.2).  (i) Giving the state that the default construction
    reaches (one step on blank from zeros) changes nothing; (ii) the predictor outputs after a given state
    follow torch.nn.LSTM started from that (h0, c0): a state that is ignored, or h and c exchanged, fails."""
    torch = pytest.importorskip("torch")
    cfg, model, enc = tiny_case(V=6, T=8, pred="lstm", seed=21, layers=2, blank_bias=1.5)
    state, o = rm.predictor_init(model)
    packed = np.stack([np.stack([state[0][l], state[1][l]]) for l in range(2)])        # [L, 2, Hd]
    args = dict(W_e=model.W_e, W_p=model.W_p, W_out=model.W_out, b_out=model.b_out, emb=model.emb,
                lstm_W_ih=model.lstm_W_ih, lstm_W_hh=model.lstm_W_hh, lstm_b=model.lstm_b)
    same = rm.RnntModel(pred_init_state=packed, **args)
    a, _ = tws.token_wise_beam_search(model, enc, 3, 2)
    b, _ = tws.token_wise_beam_search(same, enc, 3, 2)
    assert [t for t, _ in a] == [t for t, _ in b]
    np.testing.assert_allclose([x for _, x in a], [x for _, x in b], atol=1e-12)
    rng = np.random.default_rng(8)
    Hd, E = model.lstm_W_hh[0].shape[1], model.emb.shape[1]
    init = rng.standard_normal((2, 2, Hd))
    learned = rm.RnntModel(pred_init_state=init, **args)
    st0, o0 = rm.predictor_init(learned)
    np.testing.assert_array_equal(o0, init[1, 0])                                      # the top layer's h
    lib = torch.nn.LSTM(E, Hd, num_layers=2).double()
    with torch.no_grad():
        for l in range(2):
            getattr(lib, f"weight_ih_l{l}").copy_(torch.from_numpy(model.lstm_W_ih[l]))
            getattr(lib, f"weight_hh_l{l}").copy_(torch.from_numpy(model.lstm_W_hh[l]))
            getattr(lib, f"bias_ih_l{l}").copy_(torch.from_numpy(model.lstm_b[l]))
            getattr(lib, f"bias_hh_l{l}").zero_()
        tokens = [3, 1, 5]
        out, _ = lib(torch.from_numpy(model.emb[tokens]).unsqueeze(1),
                     (torch.from_numpy(init[:, 0]).unsqueeze(1).contiguous(), torch.from_numpy(init[:, 1]).unsqueeze(1).contiguous()))
    for i in range(len(tokens)):
        _, oi = rm.predictor_for_tokens(learned, tokens[:i + 1])
        np.testing.assert_allclose(oi, out[i, 0].numpy(), atol=1e-12)
    # an explicit output overrides the top layer's h for the empty prefix only
    both = rm.RnntModel(pred_init_state=init, pred_init_out=np.arange(Hd, dtype=float), **args)
    _, ob = rm.predictor_init(both)
    np.testing.assert_array_equal(ob, np.arange(Hd))
    _, o1 = rm.predictor_for_tokens(both, [3])
    np.testing.assert_allclose(o1, out[0, 0].numpy(), atol=1e-12)


def test_learned_initial_predictor_output_stateless():
    """Stateless predictor: the blank token is never a hypothesis's last token, so its embedding row serves only the
    empty prefix; a given initial output must act exactly like a model whose blank row holds that vector."""
    cfg, model, enc = tiny_case(V=6, T=8, pred="stateless", seed=22, blank_bias=1.5)
    vec = np.linspace(-1.0, 1.0, model.emb.shape[1])
    emb2 = model.emb.copy()
    emb2[model.blank] = vec
    swapped = rm.RnntModel(model.W_e, model.W_p, model.W_out, model.b_out, emb2)
    given = rm.RnntModel(model.W_e, model.W_p, model.W_out, model.b_out, model.emb, pred_init_out=vec)
    a, _ = tws.token_wise_beam_search(swapped, enc, 3, 2)
    b, _ = tws.token_wise_beam_search(given, enc, 3, 2)
    c, _ = tws.token_wise_beam_search(model, enc, 3, 2)
    assert [t for t, _ in a] == [t for t, _ in b]
    np.testing.assert_allclose([x for _, x in a], [x for _, x in b], atol=1e-12)
    assert not np.allclose([x for _, x in b][:1], [x for _, x in c][:1], atol=1e-6)     # and it does change the search


def test_stateless_predictor_is_embedding_of_last_token():
    emb = np.arange(12.0).reshape(4, 3)
    model = rm.RnntModel(np.zeros((2, 2)), np.zeros((2, 3)), np.zeros((4, 2)), np.zeros(4), emb)
    _, o = rm.predictor_init(model)
    np.testing.assert_array_equal(o, emb[0])
    _, o = rm.predictor_step(model, None, 2)
    np.testing.assert_array_equal(o, emb[2])


# ---------------------------------------------------------------- Eq. 3-7
def test_segment_math_hand_worked_golden():
    d1k1, d2k1, d1k2, d2k2, nb1, nb2, phi = _read_golden("segment_worked_example.txt")[0]
    logJ = np.log(np.array([[[0.5, 0.25, 0.25], [0.25, 0.5, 0.25]]]))
    ld_old = np.log(np.array([[0.6, 0.4]]))
    lBl = sm.blank_product(logJ)
    np.testing.assert_allclose(np.exp(lBl[0, 1, 1:4]), [1, 0.5, 0.125], atol=1e-15)
    np.testing.assert_allclose(np.exp(lBl[0, 2, 1:4]), [0, 1, 0.25], atol=1e-15)
    ld = sm.nonblank_expansion_t(logJ, lBl, ld_old)
    np.testing.assert_allclose(np.exp(ld[0, 1]), [d1k1, d2k1], atol=1e-14)
    np.testing.assert_allclose(np.exp(ld[0, 2]), [d1k2, d2k2], atol=1e-14)
    assert np.all(np.isneginf(ld[0, 0]))
    np.testing.assert_allclose(np.exp(sm.nonblank_expansion(ld)[0, 1:]), [nb1, nb2], atol=1e-14)
    np.testing.assert_allclose(np.exp(sm.blank_expansion(lBl, ld_old)), [phi], atol=1e-14)


def test_blank_product_boundary_cases():
    """Eq. 3: Bl = 1 on the diagonal, 0 below it, running product above it."""
    rng = np.random.default_rng(1)
    logJ = _random_logJ(rng, 2, 4, 5)
    lBl = sm.blank_product(logJ, blank=0)
    for t1, t2 in itertools.product(range(1, 5), range(1, 6)):
        if t1 == t2:
            assert np.all(lBl[:, t1, t2] == 0.0)
        elif t1 > t2:
            assert np.all(np.isneginf(lBl[:, t1, t2]))
        else:
            np.testing.assert_allclose(np.exp(lBl[:, t1, t2]), np.prod(np.exp(logJ[:, t1 - 1:t2 - 1, 0]), axis=1), rtol=1e-13)


@pytest.mark.parametrize("S", [1, 2, 3, 7])
def test_mass_conservation(S):
    """delta_phi + sum_{k != blank} delta_nb(k) = sum_t d_old[t] for every hypothesis."""
    rng = np.random.default_rng(S)
    H, V = 4, 9
    logJ = _random_logJ(rng, H, S, V)
    ld_old = rng.standard_normal((H, S)) * 3 - 5
    ld_old[0, 1:] = -np.inf                       # a hypothesis at segment start
    if S > 2:
        ld_old[1, 0] = -np.inf                    # no mass on the first frame
    lBl = sm.blank_product(logJ)
    ld = sm.nonblank_expansion_t(logJ, lBl, ld_old)
    total = np.logaddexp(sm.blank_expansion(lBl, ld_old), sm.logsumexp(sm.nonblank_expansion(ld)[:, 1:], axis=1))
    np.testing.assert_allclose(total, sm.logsumexp(ld_old, axis=1), rtol=0, atol=1e-12)
    # Eq. 2 / Eq. 6: the new hypothesis' score is the sum of its frame distribution
    np.testing.assert_allclose(sm.logsumexp(ld, axis=2)[:, 1:], sm.nonblank_expansion(ld)[:, 1:], atol=1e-13)


@pytest.mark.parametrize("S", [1, 2, 5, 12])
def test_explicit_sums_equal_occupancy_recursion(S):
    """a[t2] = sum_{t1<=t2} d_old[t1] Bl(t1,t2) obeys a[1] = d_old[1],
    a[t+1] = a[t] b[t] + d_old[t+1]; then d[k,t] = a[t] J(t,k) and
    delta_phi = a[S] b[S].  (This O(S) form is what a GPU scan evaluates.)"""
    rng = np.random.default_rng(10 + S)
    H, V = 3, 6
    logJ = _random_logJ(rng, H, S, V)
    d_old = np.exp(rng.standard_normal((H, S)))
    d_old[0, 1:] = 0.0
    J = np.exp(logJ)
    a = np.zeros((H, S))
    a[:, 0] = d_old[:, 0]
    for t in range(1, S):
        a[:, t] = a[:, t - 1] * J[:, t - 1, 0] + d_old[:, t]
    with np.errstate(divide="ignore"):
        ld_old = np.log(d_old)
    lBl = sm.blank_product(logJ)
    ld = sm.nonblank_expansion_t(logJ, lBl, ld_old)
    np.testing.assert_allclose(np.exp(ld[:, 1:, :]), (a[:, None, :] * np.transpose(J, (0, 2, 1)))[:, 1:, :], rtol=1e-12)
    np.testing.assert_allclose(np.exp(sm.blank_expansion(lBl, ld_old)), a[:, -1] * J[:, -1, 0], rtol=1e-12)


def test_uniform_joiner_closed_form():
    """J = 1/V everywhere, all mass on frame 1: delta_phi = V^-S and
    delta_nb(k) = sum_{t=1..S} V^-t."""
    V, S = 5, 4
    logJ = np.full((1, S, V), -math.log(V))
    ld_old = np.array([[0.0] + [-np.inf] * (S - 1)])
    lBl = sm.blank_product(logJ)
    ld = sm.nonblank_expansion_t(logJ, lBl, ld_old)
    np.testing.assert_allclose(np.exp(sm.blank_expansion(lBl, ld_old)), [V ** -S], rtol=1e-13)
    np.testing.assert_allclose(np.exp(sm.nonblank_expansion(ld)[0, 1:]), sum(V ** -t for t in range(1, S + 1)), rtol=1e-13)


def test_logsumexp_of_nothing_is_log_zero():
    assert np.isneginf(sm.logsumexp(np.array([-np.inf, -np.inf]), axis=0))
    np.testing.assert_allclose(sm.logsumexp(np.array([-np.inf, 1.0]), axis=0), 1.0)


# ---------------------------------------------------------------- list helpers
def test_add_and_merge_sums_scores_of_equal_token_sequences():
    B = []
    assert not tws.add_and_merge(B, tws.Hypothesis((1, 2), math.log(0.2), None, np.array([1.0]), None))
    assert not tws.add_and_merge(B, tws.Hypothesis((2, 1), math.log(0.1), None, np.array([2.0]), None))
    assert tws.add_and_merge(B, tws.Hypothesis((1, 2), math.log(0.3), None, np.array([9.0]), None))
    assert len(B) == 2
    assert B[0].ls == pytest.approx(math.log(0.5), abs=1e-15)
    assert B[0].o[0] == 1.0                         # first-inserted copy keeps its predictor output
    assert B[1].ls == pytest.approx(math.log(0.1))
    assert tws.choose_nth_score(B, 2) == pytest.approx(math.log(0.1))
    best = tws.choose_n_best(B, 1)
    assert best[0].tok == (1, 2)


def test_choose_n_best_expansions_order_and_ties():
    ldnb = np.log(np.array([[0.9, 0.05, 0.2, 0.2], [0.8, 0.2, 0.01, 0.3]]))
    # blank column (0) is never a candidate even though it is the largest
    assert tws.choose_n_best_expansions(ldnb, 3, blank=0) == [(1, 3), (0, 2), (0, 3)]
    assert tws.choose_n_best_expansions(ldnb, 4, blank=0)[-1] == (1, 1)
    assert len(tws.choose_n_best_expansions(ldnb, 50, blank=0)) == 6
    # the partial-sort shortcut agrees with a full sort on a large table
    rng = np.random.default_rng(5)
    big = np.round(rng.standard_normal((7, 300)), 1)    # rounded: many exact ties
    full = sorted(((-big[h, k], h, k) for h in range(7) for k in range(1, 300)))[:6]
    assert tws.choose_n_best_expansions(big, 6, blank=0) == [(h, k) for _, h, k in full]


def test_decision_log_flip_inverts_one_cut():
    log = tws.DecisionLog()
    order = tws._ordered_top([0.5, 0.1, 0.4, 0.3], 2, log, "x")
    assert order == [0, 2] and log.margins[0][2] == pytest.approx(0.1)
    assert tws._ordered_top([0.5, 0.1, 0.4, 0.3], 2, tws.DecisionLog(flips=[0]), "x") == [0, 3]
    assert log.below(0.2) == [0] and log.below(0.05) == []


# ---------------------------------------------------------------- whole algorithm
@pytest.mark.parametrize("pred,N", [("stateless", 1), ("stateless", 3), ("lstm", 2), ("lstm", 4)])
def test_segment_size_one_is_the_standard_search(pred, N):
    """S = 1 reproduces the frame-wise breadth-first search (Sec. 1, 3.2)."""
    cfg, model, enc = tiny_case(V=8, T=14, pred=pred, seed=11 + N, blank_bias=2.0)
    a, stats = tws.token_wise_beam_search(model, enc, N, 1)
    b, calls = ss.standard_beam_search(model, enc, N)
    assert [t for t, _ in a] == [t for t, _ in b]
    np.testing.assert_allclose([s for _, s in a], [s for _, s in b], atol=1e-12)
    assert stats.calls == calls


def test_segment_size_one_on_config0():
    cfg = tw_synth.get_config("c0")
    model = oracle_model(tw_synth.make_model(cfg))
    enc, _ = tw_synth.make_encoder_batch(cfg)
    a, _ = tws.token_wise_beam_search(model, enc[0], cfg.N, 1)
    b, _ = ss.standard_beam_search(model, enc[0], cfg.N)
    assert [t for t, _ in a] == [t for t, _ in b]
    np.testing.assert_allclose([s for _, s in a], [s for _, s in b], atol=1e-12)


def _all_sequences(V, U):
    for u in range(U + 1):
        yield from itertools.product(range(1, V), repeat=u)


@pytest.mark.parametrize("pred", ["stateless", "lstm"])
@pytest.mark.parametrize("T,S", [(4, 1), (4, 2), (4, 3), (4, 4), (6, 4), (5, 2), (3, 50)])
def test_unpruned_search_is_exact(pred, T, S):
    """With nothing pruned, every sequence of at most U tokens gets its exact
    RNN-T probability: forward recursion and brute-force alignment enumeration
    agree with Algorithm 1 for every segment size, including S not dividing T
    (the merge of the several routes to one sequence is part of this)."""
    V, U = 4, 2 if T > 4 else 3
    cfg, model, enc = tiny_case(V=V, T=T, pred=pred, seed=T * 10 + S)
    seqs = list(_all_sequences(V, U))
    nbest, stats = tws.token_wise_beam_search(model, enc, N=10 * len(seqs), S=S, max_len=U)
    got = dict(nbest)
    assert set(got) == set(seqs)
    for y in seqs:
        fwd = ef.forward_log_prob(model, enc, y)
        assert got[y] == pytest.approx(fwd, abs=1e-11)
        if T <= 5:
            assert ef.brute_force_log_prob(model, enc, y) == pytest.approx(fwd, abs=1e-11)
    assert stats.joins >= T


def test_forward_recursion_matches_brute_force_longer():
    cfg, model, enc = tiny_case(V=5, T=6, pred="lstm", seed=99)
    for y in [(), (1,), (3, 3), (4, 1, 2), (2, 2, 2, 2)]:
        assert ef.forward_log_prob(model, enc, y) == pytest.approx(ef.brute_force_log_prob(model, enc, y), abs=1e-11)
    # probabilities of all sequences up to some length stay below 1
    total = sum(math.exp(ef.forward_log_prob(model, enc, y)) for y in _all_sequences(5, 3))
    assert 0.0 < total < 1.0


@pytest.mark.parametrize("S", [1, 2, 3, 5, 8])
def test_pruned_scores_never_exceed_exact_probability(S):
    """Pruning only removes paths: every returned score is a lower bound of the
    sequence's exact probability, and the scores of the list sum to at most 1."""
    cfg, model, enc = tiny_case(V=6, T=10, pred="lstm", seed=5, blank_bias=1.5)
    nbest, stats = tws.token_wise_beam_search(model, enc, N=3, S=S, max_iters=4 * S + 16)
    assert len(nbest) == 3 and not stats.limit_hit
    assert [s for _, s in nbest] == sorted((s for _, s in nbest), reverse=True)
    assert len(set(t for t, _ in nbest)) == 3
    for y, s in nbest:
        assert s <= ef.forward_log_prob(model, enc, y) + 1e-10
    assert sum(math.exp(s) for _, s in nbest) <= 1.0 + 1e-12


def test_merge_of_routes_across_segments():
    """A two-token sequence reached three ways over two segments (both tokens in
    segment 1; one in each; both in segment 2) ends up as one entry whose score
    is the sum of the three path groups = the exact forward probability."""
    cfg, model, enc = tiny_case(V=3, T=4, pred="stateless", seed=21)
    nbest, _ = tws.token_wise_beam_search(model, enc, N=500, S=2, max_len=2)
    got = dict(nbest)
    y = (1, 2)
    # group the alignments of y by how many tokens fall in frames 0-1 (segment 1)
    lj = np.exp(ef._lattice_log_probs(model, enc, y))
    groups = {0: 0.0, 1: 0.0, 2: 0.0}
    for f1, f2 in itertools.product(range(4), repeat=2):
        if f1 > f2:
            continue
        p, u = 1.0, 0
        for t in range(4):
            for f in (f1, f2):
                if f == t:
                    p *= lj[t, u, y[u]]
                    u += 1
            p *= lj[t, u, 0]
        groups[(f1 < 2) + (f2 < 2)] += p
    assert all(v > 0 for v in groups.values())
    assert math.exp(got[y]) == pytest.approx(sum(groups.values()), rel=1e-11)


def test_all_blank_model_closed_form():
    """J(blank) = 1: the only hypothesis is the empty one with probability 1 and
    the joiner is called once per segment (Calls/Frame = ceil(T/S)/T)."""
    cfg, model, enc = tiny_case(V=5, T=7, pred="stateless", seed=2)
    model.W_out[:] = 0.0
    model.b_out[:] = 0.0
    model.b_out[0] = 2000.0
    for S in (1, 2, 3, 7, 9):
        nbest, stats = tws.token_wise_beam_search(model, enc, N=1, S=S, max_iters=50)
        assert nbest[0][0] == () and nbest[0][1] == pytest.approx(0.0, abs=1e-12)
        assert stats.calls == math.ceil(7 / S)
        assert stats.joins == 7


def test_uniform_model_first_segment_scores():
    """W_out = 0, b_out = 0 (uniform J), one segment covering the utterance:
    after the segment the empty hypothesis has V^-T and each single token
    sum_{t} V^-t * V^-(T-t) * ... = T * V^-(T+1)."""
    cfg, model, enc = tiny_case(V=4, T=3, pred="stateless", seed=2)
    model.W_out[:] = 0.0
    model.b_out[:] = 0.0
    nbest, _ = tws.token_wise_beam_search(model, enc, N=100, S=3, max_len=1)
    got = dict(nbest)
    assert math.exp(got[()]) == pytest.approx(4.0 ** -3, rel=1e-12)
    for k in (1, 2, 3):
        assert math.exp(got[(k,)]) == pytest.approx(3 * 4.0 ** -4, rel=1e-12)


def test_calls_per_frame_fall_and_joins_rise_with_segment_size():
    """Sec. 4.2: Calls/Frame decreases and Joins/Frame increases with S."""
    cfg = tw_synth.get_config("c0")
    model = oracle_model(tw_synth.make_model(cfg))
    enc, _ = tw_synth.make_encoder_batch(cfg)
    calls, joins = [], []
    for S in (1, 2, 4, 8):
        _, st = tws.token_wise_beam_search(model, enc[0], cfg.N, S, max_iters=4 * S + 16)
        calls.append(st.calls / st.frames)
        joins.append(st.joins / st.frames)
    assert calls == sorted(calls, reverse=True) and calls[0] > calls[-1]
    assert joins == sorted(joins) and joins[0] < joins[-1]


def test_iteration_cap_is_reported():
    cfg, model, enc = tiny_case(V=6, T=6, pred="stateless", seed=4, blank_bias=-3.0)
    _, st = tws.token_wise_beam_search(model, enc, N=2, S=3, max_iters=1)
    assert st.limit_hit and max(st.iters_per_segment) == 1


# ---- monotonic variant: every output consumes a frame ------------------------------------------------

@pytest.mark.parametrize("S", [1, 2, 3, 7])
def test_monotonic_mass_conservation_and_shift(S):
    """Monotonic segment formulas: mass is conserved (including what has already left the segment), a new
    hypothesis sits one frame after its emission, and delta_nb equals the standard one on the same input."""
    rng = np.random.default_rng(40 + S)
    H, V = 4, 7
    logJ = _random_logJ(rng, H, S, V)
    ld_old = rng.standard_normal((H, S + 1)) * 3 - 5
    ld_old[0, 1:] = -np.inf                       # a hypothesis at segment start
    ld_old[1, :S] = -np.inf                       # a hypothesis that has left the segment entirely
    lBl = sm.blank_product(logJ)
    ld = sm.nonblank_expansion_t_monotonic(logJ, lBl, ld_old)
    dphi = sm.blank_expansion_monotonic(lBl, ld_old)
    total = np.logaddexp(dphi, sm.logsumexp(sm.nonblank_expansion(ld)[:, 1:], axis=1))
    np.testing.assert_allclose(total, sm.logsumexp(ld_old, axis=1), rtol=0, atol=1e-12)
    assert np.all(np.isneginf(ld[:, :, 0]))       # nothing can sit on the first frame after an emission
    std = sm.nonblank_expansion_t(logJ, lBl, ld_old[:, :S])
    np.testing.assert_allclose(ld[:, 1:, 1:], std[:, 1:, :], atol=1e-13)
    assert dphi[1] == pytest.approx(ld_old[1, S], abs=1e-13) and np.all(np.isneginf(ld[1]))
    np.testing.assert_allclose(np.exp(dphi), np.exp(sm.blank_expansion(lBl, ld_old[:, :S])) + np.exp(ld_old[:, S]), rtol=1e-12)


@pytest.mark.parametrize("pred", ["stateless", "lstm"])
@pytest.mark.parametrize("T,S", [(4, 1), (4, 2), (4, 3), (4, 4), (6, 4), (5, 2), (3, 50)])
def test_monotonic_unpruned_search_is_exact(pred, T, S):
    """Un-pruned, the monotonic search gives every sequence of at most T tokens the sum over all placements
    of its tokens on distinct frames: forward recursion and brute force agree, for every segment size."""
    V, U = 4, 3
    cfg, model, enc = tiny_case(V=V, T=T, pred=pred, seed=T * 10 + S + 500)
    seqs = [y for y in _all_sequences(V, U) if len(y) <= T]
    nbest, stats = tws.token_wise_beam_search(model, enc, N=10 * len(seqs) + 10, S=S, max_len=U, monotonic=True)
    got = dict(nbest)
    assert set(seqs) <= set(got)
    for y in seqs:
        fwd = ef.forward_log_prob_monotonic(model, enc, y)
        assert got[y] == pytest.approx(fwd, abs=1e-11)
        assert ef.brute_force_log_prob_monotonic(model, enc, y) == pytest.approx(fwd, abs=1e-11)
    # a monotonic model spreads all its mass over sequences of at most T tokens
    if U >= T:
        assert sum(math.exp(s) for s in got.values()) == pytest.approx(1.0, abs=1e-10)
    # it is a different lattice from the standard one: the same sequence gets a different probability
    assert abs(got[(1, 1)] - ef.forward_log_prob(model, enc, (1, 1))) > 1e-6


@pytest.mark.parametrize("pred,N", [("stateless", 1), ("stateless", 3), ("lstm", 2), ("lstm", 4)])
def test_monotonic_segment_size_one_is_the_frame_synchronous_search(pred, N):
    cfg, model, enc = tiny_case(V=6, T=9, pred=pred, seed=21 + N, blank_bias=1.0)
    ref = ss.monotonic_frame_search(model, enc, N)
    got, stats = tws.token_wise_beam_search(model, enc, N=N, S=1, monotonic=True)
    assert [t for t, _ in got] == [t for t, _ in ref]
    np.testing.assert_allclose([s for _, s in got], [s for _, s in ref], atol=1e-12)
    assert all(len(t) <= 9 for t, _ in got)


@pytest.mark.parametrize("S", [2, 3, 5, 8])
def test_monotonic_pruned_scores_never_exceed_exact_probability(S):
    cfg, model, enc = tiny_case(V=6, T=10, pred="lstm", seed=5, blank_bias=1.5)
    nbest, stats = tws.token_wise_beam_search(model, enc, N=3, S=S, max_iters=4 * S + 16, monotonic=True)
    assert len(nbest) == 3 and not stats.limit_hit
    for y, s in nbest:
        assert s <= ef.forward_log_prob_monotonic(model, enc, y) + 1e-10
    assert max(stats.iters_per_segment) <= S + 1     # at most one token per frame, then everything has left


# ---- blank thresholding on a factorised output (Sec. 2, Sec. 5; the rule is this build's reading) ----------------
def _hat_case(**kw):
    cfg, model, enc = tiny_case(**kw)
    hat = rm.RnntModel(model.W_e, model.W_p, model.W_out, model.b_out, model.emb, model.lstm_W_ih, model.lstm_W_hh,
                       model.lstm_b, normalisation="hat")
    return cfg, hat, enc


def test_hat_output_hand_worked_golden():
    rows = _read_golden("hat_closed_form.txt")
    z1 = np.array([np.log(3.0), 0.0, np.log(2.0)])
    z2 = np.array([np.log(2.0), -np.log(4.0), 0.0])
    np.testing.assert_allclose(np.exp(rm.log_hat(z1[None], 0))[0], rows[0], atol=1e-12)
    np.testing.assert_allclose(np.exp(rm.log_hat(z2[None], 1))[0], rows[1], atol=1e-12)
    # through the joiner: a distribution per (hypothesis, frame), blank probability = sigmoid of the blank logit
    cfg, hat, enc = _hat_case(V=6, T=5, pred="lstm", seed=3)
    _, o = rm.predictor_init(hat)
    lj = rm.joiner_log_probs(hat, enc, o[None])
    np.testing.assert_allclose(np.exp(lj).sum(axis=-1), 1.0, atol=1e-12)
    soft = rm.RnntModel(hat.W_e, hat.W_p, hat.W_out, hat.b_out, hat.emb, hat.lstm_W_ih, hat.lstm_W_hh, hat.lstm_b)
    ls = rm.joiner_log_probs(soft, enc, o[None])
    # same logits underneath: ratios between non-blank tokens are those of the plain softmax
    np.testing.assert_allclose(lj[..., 2] - lj[..., 3], ls[..., 2] - ls[..., 3], atol=1e-12)
    # and the blank probability is the logistic function of the blank logit itself
    z0 = np.tanh(enc @ hat.W_e.T + o @ hat.W_p.T) @ hat.W_out[0] + hat.b_out[0]
    np.testing.assert_allclose(np.exp(lj[0, :, 0]), 1.0 / (1.0 + np.exp(-z0)), atol=1e-12)


def test_blank_threshold_rule_on_a_table():
    logJ = np.log(np.array([[[0.7, 0.2, 0.1], [0.4, 0.5, 0.1]], [[0.95, 0.03, 0.02], [0.6, 0.3, 0.1]]]))
    out, skip = rm.apply_blank_threshold(logJ, 0.65, 0)
    assert skip.tolist() == [[True, False], [True, False]]
    np.testing.assert_allclose(np.exp(out[0, 0]), [0.7, 0.0, 0.0], atol=1e-15)
    np.testing.assert_allclose(np.exp(out[0, 1]), [0.4, 0.5, 0.1], atol=1e-15)
    np.testing.assert_allclose(np.exp(out[1, 0]), [0.95, 0.0, 0.0], atol=1e-15)
    same, none = rm.apply_blank_threshold(logJ, 1.0, 0)
    assert not none.any() and np.array_equal(same, logJ)
    allb, every = rm.apply_blank_threshold(logJ, 0.0, 0)
    assert every.all() and np.all(np.isneginf(allb[..., 1:])) and np.array_equal(allb[..., 0], logJ[..., 0])


@pytest.mark.parametrize("pred", ["stateless", "lstm"])
@pytest.mark.parametrize("T,S,tau", [(4, 1, 1.0), (4, 2, 1.0), (4, 3, 0.5), (5, 2, 0.35), (4, 4, 0.6), (6, 4, 0.45), (3, 50, 0.5)])
def test_unpruned_search_with_blank_threshold_is_exact(pred, T, S, tau):
    """Nothing pruned: every sequence gets exactly the sum over its alignments on the thresholded lattice (nodes
    whose blank probability exceeds the threshold keep their blank arc only), for every segment size.  tau = 1 is
    plain Algorithm 1 on the factorised distribution."""
    V, U = 4, 2 if T > 4 else 3
    cfg, hat, enc = _hat_case(V=V, T=T, pred=pred, seed=T * 10 + S, blank_bias=0.0)
    seqs = list(_all_sequences(V, U))
    nbest, stats = tws.token_wise_beam_search(hat, enc, N=10 * len(seqs), S=S, max_len=U, blank_threshold=tau)
    got = dict(nbest)
    assert stats.skipped == 0 or tau < 1.0
    for y in seqs:
        with np.errstate(divide="ignore"):
            fwd = ef.forward_log_prob(hat, enc, y, blank_threshold=tau)
            brute = ef.brute_force_log_prob(hat, enc, y, blank_threshold=tau) if T <= 5 else fwd
        if np.isneginf(fwd):
            assert y not in got or np.isneginf(got[y])
            continue
        assert got[y] == pytest.approx(fwd, abs=1e-11)
        assert brute == pytest.approx(fwd, abs=1e-11)
    assert stats.frame_rows >= stats.joins and stats.skipped <= stats.frame_rows


def test_blank_threshold_zero_keeps_only_the_empty_hypothesis():
    """Threshold 0: every frame is skipped, no token is ever emitted, and the score is the product of the blank
    probabilities of the empty prefix along the utterance."""
    cfg, hat, enc = _hat_case(V=6, T=9, pred="lstm", seed=12)
    nbest, stats = tws.token_wise_beam_search(hat, enc, 3, 4, blank_threshold=0.0)
    _, o = rm.predictor_init(hat)
    lj = rm.joiner_log_probs(hat, enc, o[None])[0]
    assert [t for t, _ in nbest] == [()]
    assert nbest[0][1] == pytest.approx(lj[:, 0].sum(), abs=1e-12)
    assert stats.skipped == stats.frame_rows == 9 and stats.calls == 3


def test_blank_threshold_mass_accounting():
    """delta_phi + sum_k delta_nb + (mass of the label parts left out) = sum_t d_old, with the left-out mass written
    as the explicit sum over the skipped frames t2 of sum_{t1 <= t2} d_old(t1) Bl(t1, t2) (1 - J(t2, blank))."""
    rng = np.random.default_rng(5)
    H, S, V = 3, 4, 7
    logJ = rm.log_hat(rng.standard_normal((H, S, V)) * 2.0, 0)
    ld_old = rng.standard_normal((H, S)) - 1.0
    thr, skip = rm.apply_blank_threshold(logJ, 0.4, 0)
    assert skip.any() and not skip.all()
    lBl = sm.blank_product(thr)
    ld = sm.nonblank_expansion_t(thr, lBl, ld_old)
    nb = np.exp(sm.nonblank_expansion(ld))[:, 1:].sum(axis=1)
    phi = np.exp(sm.blank_expansion(lBl, ld_old))
    left_out = np.zeros(H)
    for h in range(H):
        for t2 in range(1, S + 1):
            if skip[h, t2 - 1]:
                a = sum(np.exp(ld_old[h, t1 - 1] + lBl[h, t1, t2]) for t1 in range(1, t2 + 1))
                left_out[h] += a * (1.0 - np.exp(logJ[h, t2 - 1, 0]))
    np.testing.assert_allclose(phi + nb + left_out, np.exp(ld_old).sum(axis=1), rtol=1e-12)

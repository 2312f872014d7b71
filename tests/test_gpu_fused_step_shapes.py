"""The fused joiner kernel (joiner + softmax + Eq. 3-7 with the logits in tensor memory) at the row counts of
the timed decode steps, element by element against the fp64 oracle.

A cluster owns a row tile; with more tiles than resident clusters every cluster walks several tiles: the
second accumulator buffer, the wrap of the accumulator phase at the third tile, the operand ring running on
across tiles, the prefetch of the cluster's next tile and a ragged last round.  Every delta_phi, delta_nb and
occupancy value of every row is compared with oracle.segment_math on oracle.rnnt_model.joiner_log_probs at
the bf16 stage tolerance."""
import numpy as np
import pytest

import tw_synth
from oracle import rnnt_model as rm
from oracle import segment_math as sm
from helpers import oracle_model

pytestmark = pytest.mark.gpu
BF16_STAGE_TOL = 2e-2


def _oracle_rows(om, enc, pred, ld_old, row_group, seg_len, V):
    """(delta_phi [R], delta_nb [R, V], occupancy la [R, S]) from the oracle, segment by segment."""
    R, S = ld_old.shape
    phi = np.empty(R)
    nb = np.empty((R, V))
    la = np.full((R, S), -np.inf)
    for g in np.unique(row_group):
        rows = np.nonzero(row_group == g)[0]
        sl = int(seg_len[g])
        lj = rm.joiner_log_probs(om, enc[g, :sl], pred[rows])                # [H, sl, V]
        lo = ld_old[rows, :sl].astype(np.float64)
        lBl = sm.blank_product(lj, om.blank)
        ld = sm.nonblank_expansion_t(lj, lBl, lo, om.blank)                   # [H, V, sl]
        nb[rows] = sm.nonblank_expansion(ld)
        phi[rows] = sm.blank_expansion(lBl, lo)
        k = 1 if om.blank != 1 else 2                                        # Eq. 5: log d(k, t) = la[t] + log J(t, k)
        with np.errstate(invalid="ignore"):
            la_g = ld[:, k, :] - lj[:, :, k]
        la[rows, :sl] = np.where(np.isneginf(ld[:, k, :]), -np.inf, la_g)
    return phi, nb, la


def _compare(got, ref, seg_len_row, blank, what):
    phi, nb, la = got
    rphi, rnb, rla = ref
    R, V = nb.shape
    assert np.all(np.isfinite(phi)), what
    assert np.abs(phi - rphi).max() < BF16_STAGE_TOL, (what, "delta_phi", np.abs(phi - rphi).max())
    assert np.all(np.isneginf(nb[:, blank])), what
    cols = np.arange(V) != blank
    assert np.all(np.isfinite(nb[:, cols])), (what, "delta_nb has log 0 where the oracle has mass")
    err = np.abs(nb[:, cols] - rnb[:, cols])
    worst = np.unravel_index(np.argmax(err), err.shape)
    assert err.max() < BF16_STAGE_TOL, (what, "delta_nb", err.max(), "row %d" % worst[0])
    inf_g, inf_r = np.isneginf(la), np.isneginf(rla)
    assert np.array_equal(inf_g, inf_r), (what, "occupancy: log 0 pattern")
    assert np.abs(la[~inf_r] - rla[~inf_r]).max() < BF16_STAGE_TOL, (what, "occupancy")
    for r in range(R):
        assert np.all(inf_g[r, seg_len_row[r]:])


def _fix_dead_rows(ld_old, seg_len_row):
    for r in range(ld_old.shape[0]):
        if not np.any(np.isfinite(ld_old[r, :seg_len_row[r]])):
            ld_old[r, 0] = -1.0


def _run(cfg, S, N, R, G, seed, min_rounds=3):
    from paper_2302_14357_b200.binding import MODE_BF16, TwDecoder, weights_from_synth
    m = tw_synth.make_model(cfg)
    max_batch = (R + N - 1) // N
    dec = TwDecoder(weights_from_synth(m), N=N, S=S, mode=MODE_BF16, max_batch=max_batch,
                    max_T=max(8, (G * S + max_batch - 1) // max_batch), joiner_act=cfg.joiner_act)   # room for G * S frames
    assert dec.set_fused(True)
    st = dec.stats()
    HPT = 4 * (32 // S)
    tiles = (R + HPT - 1) // HPT
    clusters = st["fused_clusters"]
    assert clusters >= 1
    # the point of these sizes: at least three tiles per cluster and a last round that is not full
    assert tiles >= min_rounds * clusters and tiles % clusters != 0, (tiles, clusters)
    om = oracle_model(m)
    rng = np.random.default_rng(seed)
    enc = tw_synth.round_to_bf16(rng.standard_normal((G, S, cfg.D_enc)).astype(np.float32))
    row_group = np.sort(rng.integers(0, G, size=R)).astype(np.int32)          # a segment's hypotheses are neighbours
    seg_len = rng.integers(1, S + 1, size=G).astype(np.int32)
    seg_len[rng.random(G) < 0.7] = S
    pred = (rng.standard_normal((R, cfg.P)) * 0.5).astype(np.float32)
    ld_old = (rng.standard_normal((R, S)) * 1.5 - 2).astype(np.float32)
    kind = rng.integers(0, 4, size=R)
    ld_old[kind == 0, 1:] = -np.inf                                          # segment start: all mass on frame 1
    if S > 1:
        ld_old[kind == 1, 0] = -np.inf                                       # no mass left on frame 1
    _fix_dead_rows(ld_old, seg_len[row_group])
    E = dec.project_encoder(enc).reshape(G, S, cfg.J)
    Pp = (pred.astype(np.float64) @ om.W_p.T).astype(np.float32)            # input marshalling only
    got = [x.cpu().numpy().astype(np.float64) for x in dec.joiner_expand(E, Pp, row_group, seg_len, ld_old)]
    # twice in a row on the same handle: barrier phases and buffers start afresh in every launch
    again = [x.cpu().numpy().astype(np.float64) for x in dec.joiner_expand(E, Pp, row_group, seg_len, ld_old)]
    for a, b in zip(got, again):
        np.testing.assert_array_equal(a, b)
    dec.close()
    ref = _oracle_rows(om, enc, pred, ld_old, row_group, seg_len, cfg.V)
    _compare(got, ref, seg_len[row_group], om.blank, "%s S=%d R=%d" % (cfg.name, S, R))


def test_fused_joiner_c3_step_shape_every_element():
    """B = 128 utterances x N = 10 hypotheses, S = 3, V = 4096, J = 1024: 32 row tiles of 40 hypotheses on the 7
    resident clusters of 16 CTAs, five tiles for some clusters and four for others."""
    cfg = tw_synth.get_config("c3")
    _run(cfg, S=3, N=10, R=1275, G=128, seed=31)


def test_fused_joiner_two_frame_segments_every_element():
    """S = 2 on the c3 model: 64 hypotheses per tile, 24 tiles on the 7 resident clusters (the two lanes of a
    hypothesis share out the columns of delta_nb between them)."""
    cfg = tw_synth.get_config("c3")
    _run(cfg, S=2, N=10, R=1500, G=150, seed=36)


def test_fused_joiner_c4_step_shape_every_element():
    """S = 10 (the staged sums over a hypothesis's frames), V = 4096, J = 1024, 2590 rows: 216 tiles of 12
    hypotheses, 31 rounds on 7 clusters, the last one ragged."""
    cfg = tw_synth.get_config("c4")
    _run(cfg, S=10, N=10, R=2590, G=259, seed=32)


@pytest.mark.parametrize("S,R", [(5, 2810), (8, 1900)])
def test_fused_joiner_librispeech_shape_long_segments_every_element(S, R):
    """V = 1024, J = 640 (clusters of 4 CTAs, 37 resident): S = 5 and S = 8 take the staged-sum epilogue."""
    cfg = tw_synth.get_config("c2")
    _run(cfg, S=S, N=16, R=R, G=R // 12, seed=33 + S)


@pytest.mark.parametrize("S,R,rounds", [(3, 2650, 0), (5, 6000, 3)])
def test_fused_joiner_padded_vocabulary_every_element(S, R, rounds):
    """V = 501 (padded to 512 columns for the kernel, clusters of 2 CTAs, 74 resident) with the ReLU joiner of
    the paper's models (Sec. 4.1): the stage returns the 501 real columns.  One tile per cluster, and four."""
    cfg = tw_synth.get_config("p1")
    _run(cfg, S=S, N=16, R=R, G=R // 10, seed=40 + S, min_rounds=rounds)

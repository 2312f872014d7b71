"""tw_joiner_expand_noalloc: the handle-free, allocation-free packaging of the joiner + expansion
stage, meant for processes whose device memory is owned by another allocator.  It must give what
tw_joiner_expand gives, call after call, although all calls share one fixed scratch array that still
holds the previous call's data.  Collected last on purpose."""
import numpy as np
import pytest

import tw_synth

pytestmark = pytest.mark.gpu


def _case(rng, cfg, S, G, R):
    E = rng.standard_normal((G, S, cfg.J)).astype(np.float32)
    Pp = rng.standard_normal((R, cfg.J)).astype(np.float32)
    row_group = rng.integers(0, G, size=R).astype(np.int32)
    seg_len = rng.integers(1, S + 1, size=G).astype(np.int32)
    ld_old = (rng.standard_normal((R, S)) - 2).astype(np.float32)
    ld_old[0, 1:] = -np.inf
    return E, Pp, row_group, seg_len, ld_old


def test_noalloc_entry_point_matches_handle_path_twice_in_a_row():
    import torch
    from paper_2302_14357_b200 import binding
    cfg = tw_synth.WorkloadConfig("na", 4, 16, (16, 16), 24, "stateless", 20, 0, 0, 40, 150, 2.0, 3, (5,), "f32", 17)
    S = 5
    m = tw_synth.make_model(cfg)
    dec = binding.TwDecoder(binding.weights_from_synth(m), N=3, S=S, max_batch=8, max_T=16)
    W_out = torch.from_numpy(m.W_out).cuda()
    b_out = torch.from_numpy(m.b_out).cuda()
    rng = np.random.default_rng(5)
    # second call is smaller than the first: the scratch still holds the first call's rows
    for G, R in ((4, 21), (2, 6)):
        E, Pp, row_group, seg_len, ld_old = [torch.from_numpy(x).cuda() for x in _case(rng, cfg, S, G, R)]
        ref = dec.joiner_expand(E, Pp, row_group, seg_len, ld_old)
        st, ldphi, ldnb, la = binding.joiner_expand_noalloc(W_out, b_out, S, 0, E, Pp, row_group, seg_len, ld_old)
        torch.cuda.synchronize()
        assert st == 0
        for got, want in zip((ldphi, ldnb, la), ref):
            got, want = got.cpu().numpy(), want.cpu().numpy()
            assert np.array_equal(np.isneginf(got), np.isneginf(want))
            fin = np.isfinite(want)
            np.testing.assert_allclose(got[fin], want[fin], rtol=1.2e-7, atol=1e-5)
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

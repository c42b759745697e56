"""Sampling-based acceptance on the GPU (Sec. 2.2, Eq. 1) against the oracle: `cass_softmax`, `cass_sample` and
`cass_accept_sampling` through the C boundary.  Random numbers are inputs on both sides."""
import numpy as np
import pytest
import torch

import synth
from oracle import model

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def cass():
    import paper_2605_26558_b200 as m
    from paper_2605_26558_b200 import engine
    m.engine = engine
    return m


def _valid_draw(weights64, u, pick, slack=2e-5):
    """An inverse-CDF pick is the lowest index whose cumulative weight exceeds u * total.  The GPU sums in fp32 in
    another order, so a pick is accepted when it satisfies that definition for some threshold within `slack` (relative
    to the total) of u * total, and it must never land on an index of zero weight."""
    c = np.cumsum(weights64)
    tot = c[-1]
    lo = c[pick - 1] if pick > 0 else 0.0
    return weights64[pick] > 0 and lo <= u * tot + slack * tot and c[pick] >= u * tot - slack * tot


@pytest.mark.parametrize("rows,vocab,temp", [(3, 16, 1.0), (5, 1000, 0.7), (2, 128256, 1.3)])
def test_softmax_and_sample(cass, rows, vocab, temp):
    g = torch.Generator().manual_seed(vocab)
    logits = (torch.randn(rows, vocab, generator=g) * 3).cuda()
    probs = torch.zeros(rows, vocab, dtype=torch.float32, device="cuda")
    cass.cass_softmax(logits, rows, vocab, temp, probs)
    want = np.stack([model.softmax(logits[r].cpu().numpy(), temp) for r in range(rows)])
    got = probs.cpu().numpy().astype(np.float64)
    assert np.allclose(got, want, rtol=2e-5, atol=1e-9)
    assert np.allclose(got.sum(1), 1.0, atol=1e-5)
    for trial in range(6):
        u = torch.rand(rows, generator=g)
        if trial == 0:
            u[0] = 0.0
        toks = torch.full((rows * 2,), -1, dtype=torch.int32, device="cuda")
        cass.cass_sample(probs, rows, vocab, u.cuda(), toks, tok_stride=2)
        t = toks.cpu().numpy()
        for r in range(rows):
            pick = int(t[2 * r])
            assert 0 <= pick < vocab and t[2 * r + 1] == -1
            assert _valid_draw(got[r], float(u[r]), pick), (r, pick)
            want_pick = model.inverse_cdf_sample(got[r], float(u[r]))
            c = np.cumsum(got[r])
            margin = min(abs(c[want_pick] - float(u[r]) * c[-1]), abs((c[want_pick - 1] if want_pick else 0.0) - float(u[r]) * c[-1]))
            if margin > 1e-4:                      # away from a boundary the pick is unique
                assert pick == want_pick


def test_accept_sampling_against_the_oracle_and_in_distribution(cass):
    """100 000 independent 'sequences' (no session): 16-symbol vocabulary, gamma = 3.  n equals Eq. 1 evaluated by the
    oracle, the emitted tokens are the oracle's (or, at a cumulative-sum boundary, a valid draw), and the first
    emitted token is distributed as the target's first distribution (chi-square, 15 degrees of freedom)."""
    rng = np.random.default_rng(0)
    N, V, g = 100_000, 16, 3
    p1 = rng.dirichlet(np.ones(V) * 0.7, size=g + 1).astype(np.float32)
    q1 = rng.dirichlet(np.ones(V) * 0.7, size=g).astype(np.float32)
    q1[1, 5] = 0.0                                  # a token the draft cannot emit but the target can
    q1[1] /= q1[1].sum()
    p = np.broadcast_to(p1, (N, g + 1, V)).copy()
    q = np.broadcast_to(q1, (N, g, V)).copy()
    drafts = np.stack([rng.choice(V, size=N, p=q1[i].astype(np.float64) / q1[i].astype(np.float64).sum()) for i in range(g)], axis=1).astype(np.int32)
    r = rng.uniform(size=(N, g)).astype(np.float32)
    u = rng.uniform(size=N).astype(np.float32)
    n_acc = torch.full((N,), -1, dtype=torch.int32, device="cuda")
    out = torch.full((N, g + 1), -9, dtype=torch.int32, device="cuda")
    nxt = torch.full((N,), -9, dtype=torch.int32, device="cuda")
    cass.cass_accept_sampling(None, N, torch.from_numpy(drafts).cuda(), torch.from_numpy(p).cuda(), torch.from_numpy(q).cuda(), V,
                              torch.from_numpy(r).cuda(), torch.from_numpy(u).cuda(), g, n_acc, out, nxt)
    torch.cuda.synchronize()
    n_got, out_got, nxt_got = n_acc.cpu().numpy(), out.cpu().numpy(), nxt.cpu().numpy()
    first = np.zeros(V)
    boundary = 0
    for i in range(N):
        n, toks = model.sampling_accept(p1, q1, drafts[i].tolist(), r[i], float(u[i]))
        x = drafts[i]
        margins = [abs(float(r[i, j]) * float(q1[j, x[j]]) - float(p1[j, x[j]])) for j in range(min(n + 1, g))]
        if min(margins + [1.0]) < 1e-6:             # r * q == p to rounding: either decision is right
            continue
        assert n_got[i] == n, i
        assert out_got[i, :n].tolist() == toks[:n] and (out_got[i, n + 1:] == -1).all()
        extra = int(out_got[i, n])
        assert nxt_got[i] == extra
        if extra != toks[n]:
            w = np.maximum(p1[n].astype(np.float64) - q1[n].astype(np.float64), 0.0) if n < g else p1[g].astype(np.float64)
            assert _valid_draw(w, float(u[i]), extra), i
            boundary += 1
        first[out_got[i, 0]] += 1
    assert boundary < N * 1e-3
    exp = p1[0].astype(np.float64) / p1[0].astype(np.float64).sum() * first.sum()
    assert float(((first - exp) ** 2 / exp).sum()) < 37.7


def test_accept_sampling_special_cases_and_session_lengths(cass):
    """One-hot distributions reduce Eq. 1 to the greedy rule; identical models accept everything; with a session the
    committed lengths move by n + 1 as after cass_accept."""
    shape = synth.TINY
    wt = synth.model_weights(shape, 0, device="cuda")
    gw = {"layers": [cass.engine.fuse_layer_weights(lw) for lw in wt["layers"]], "embed": wt["embed"], "lm_head": wt["lm_head"],
          "norm_final": wt["norm_final"]}
    eng = cass.engine.Engine(shape, gw, max_seq=128, gamma_max=4, batch=2)
    V, g = shape.vocab, 3
    tgt = np.array([[3, 5, 1, 7], [10, 11, 12, 13]])
    drf = np.array([[3, 5, 2], [10, 11, 12]], dtype=np.int32)
    eye = np.eye(V, dtype=np.float32)
    p = np.stack([eye[tgt[b]] for b in range(2)])
    q = np.stack([eye[drf[b]] for b in range(2)])
    cass.cass_set_lens(eng.session, [20, 30] + [0] * 6)
    n_acc = torch.zeros(8, dtype=torch.int32, device="cuda")
    out = torch.zeros(2 * (g + 1), dtype=torch.int32, device="cuda")
    nxt = torch.zeros(2, dtype=torch.int32, device="cuda")
    r = torch.full((2, g), 0.5, device="cuda")
    u = torch.tensor([0.3, 0.9], device="cuda")
    cass.cass_accept_sampling(eng.session, 2, torch.from_numpy(drf).cuda(), torch.from_numpy(p).cuda(), torch.from_numpy(q).cuda(),
                              V, r, u, g, n_acc, out, nxt)
    torch.cuda.synchronize()
    assert n_acc[:2].tolist() == [model.greedy_accept(drf[b].tolist(), tgt[b].tolist()) for b in range(2)] == [2, 3]
    assert out.view(2, g + 1).tolist() == [[3, 5, 1, -1], [10, 11, 12, 13]] and nxt.tolist() == [1, 13]
    assert eng.lens() == [23, 34] and eng.status()[0] == 0
    with pytest.raises(cass.CassError):                # a session takes exactly its own number of sequences
        cass.cass_accept_sampling(eng.session, 1, torch.from_numpy(drf).cuda(), torch.from_numpy(p).cuda(),
                                  torch.from_numpy(q).cuda(), V, r, u, g, n_acc, out, nxt)
    eng.close()

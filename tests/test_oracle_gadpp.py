"""Pins of the checker's relaxed verification (Section 3.2.3 of the paper, Eq. 8 and Eq. 9): brute force on
random scores, the literal log-likelihood form, the two limits the section implies (beta = 1 with tau = 0 is the
exact-match verification; beta = V with an unbounded tau keeps every draft), monotonicity in beta and tau, and a
whole-loop invariant (every output token is the greedy choice or meets the requirement given its prefix).
The section's own numbers (block-size and beta/tau sweeps) need the trained models: parity unpinned there."""
import numpy as np
import pytest

from oracle import ad_oracle as O
from paper_2205_10350_b200 import synth

OPS = O.Ops("f32")
OPS64 = O.Ops("f64")


def _brute(lg, d, beta, tau):
    """Independent statement of the two conditions: fewer than beta tokens score strictly higher than the draft
    (so its score is at least the beta-th ranked one), and the best score exceeds it by at most tau."""
    if d < 0:
        return False
    higher = int((lg > lg[d]).sum())
    return higher <= beta - 1 and float(lg.max()) - float(lg[d]) <= tau


def test_relaxed_choice_brute_force_random_scores():
    r = np.random.default_rng(5)
    for trial in range(600):
        V = int(r.integers(2, 40))
        lg = r.normal(size=V).astype(np.float32)
        if trial % 3 == 0:                                  # integer scores: plenty of exact ties
            lg = r.integers(0, 4, size=V).astype(np.float32)
        d = int(r.integers(-1, V))
        beta = int(r.integers(1, V + 3))
        tau = float(r.choice([0.0, 0.3, 1.0, 2.5, 1e30]))
        tok, met, tm, dm = OPS.relaxed_choice(lg, d, beta, tau)
        want = _brute(lg, d, beta, tau)
        assert met == want, (lg, d, beta, tau)
        assert tok == (d if want else int(np.argmax(lg)))   # numpy's argmax also takes the lowest index on ties
        srt = np.sort(lg)[::-1]
        assert tm == pytest.approx(srt[0] - srt[1])


def test_relaxed_choice_is_the_log_likelihood_form():
    """Eq. 8 and Eq. 9 are stated on log P; evaluate them literally with a float64 log-softmax."""
    r = np.random.default_rng(6)
    for _ in range(300):
        V = 50
        lg = (r.normal(size=V) * 2).astype(np.float64)
        d = int(r.integers(0, V))
        beta = int(r.integers(1, 8))
        tau = float(r.uniform(0, 3))
        logp = lg - np.log(np.exp(lg - lg.max()).sum()) - lg.max()
        ranked = np.sort(logp)[::-1]
        want = logp[d] >= ranked[beta - 1] and ranked[0] - logp[d] <= tau
        tok, met, _, dm = OPS64.relaxed_choice(lg, d, beta, tau)
        if dm > 1e-9:                                       # away from a knife edge the two forms must agree
            assert met == bool(want)


def test_decision_margin_bounds_the_distance_to_a_flip():
    """Moving the draft's score by less than the reported margin never changes the decision (the margin is the
    distance to the nearer of the two thresholds; crossing it flips the decision whenever the other condition
    does not decide alone, which must happen often on random scores)."""
    r = np.random.default_rng(7)
    flips = 0
    for _ in range(300):
        V = 30
        lg = r.normal(size=V).astype(np.float64)
        d = int(r.integers(0, V))
        if d == int(np.argmax(lg)):
            continue
        beta, tau = int(r.integers(1, 6)), float(r.uniform(0.1, 2.0))
        _, met, _, dm = OPS64.relaxed_choice(lg, d, beta, tau)
        assert np.isfinite(dm)
        for sign in (-1.0, 1.0):
            near = lg.copy(); near[d] += sign * 0.9 * dm
            if int(np.argmax(near)) == int(np.argmax(lg)):
                assert OPS64.relaxed_choice(near, d, beta, tau)[1] == met
        far_dn = lg.copy(); far_dn[d] -= 1.1 * dm
        far_up = lg.copy(); far_up[d] += 1.1 * dm
        if int(np.argmax(far_up)) == int(np.argmax(lg)):
            changed = (OPS64.relaxed_choice(far_dn, d, beta, tau)[1] != met) or (OPS64.relaxed_choice(far_up, d, beta, tau)[1] != met)
            flips += changed
    assert flips > 50


@pytest.fixture(scope="module")
def tiny():
    m = O.Model(synth.TINY, synth.make_weights(synth.TINY, 0), max_pos=64)
    src, lens = synth.make_sources(synth.WORKLOADS[1])
    st = m.state(src[0, :lens[0]])
    g, _ = st.greedy(24)
    return m, st, g


def _drafts(st, g, k, r):
    """A block whose drafts are a mix of the greedy token, a runner-up of the true scores and noise."""
    st.reset()
    lg = st.verify_block(0, g[:k], want_logits=True)["logits"]
    d = g[:k].copy()
    for i in range(k):
        u = r.random()
        order = np.argsort(-lg[i], kind="stable")
        if u < 0.35:
            d[i] = order[int(r.integers(1, 6))]
        elif u < 0.5:
            d[i] = int(r.integers(4, lg.shape[1]))
    return d.astype(np.int32)


def test_beta_one_tau_zero_is_exact_match(tiny):
    m, st, g = tiny
    r = np.random.default_rng(8)
    for _ in range(6):
        d = _drafts(st, g, 12, r)
        st.reset()
        a = st.verify_block(0, d)
        st.reset()
        b = st.verify_block_pp(0, d, 1, 0.0)
        assert np.array_equal(a["pred"], b["pred"]) and a["n"] == b["n"] and a["finished"] == b["finished"]
        assert np.array_equal(b["met"], d == a["pred"])


def test_unbounded_requirement_keeps_every_draft(tiny):
    m, st, g = tiny
    r = np.random.default_rng(9)
    d = _drafts(st, g, 12, r)
    d[d == 2] = 5                                           # no [EOS] among the drafts
    st.reset()
    b = st.verify_block_pp(0, d, synth.TINY.vocab, 1e30)
    assert b["met"].all() and np.array_equal(b["pred"], d) and b["n"] == len(d) and not b["finished"]
    d[-1] = -1                                              # a sentinel slot never qualifies
    st.reset()
    b = st.verify_block_pp(0, d, synth.TINY.vocab, 1e30)
    assert not b["met"][-1] and b["n"] == len(d)


def test_accepted_length_is_monotone_in_beta_and_tau(tiny):
    m, st, g = tiny
    r = np.random.default_rng(10)
    betas, taus = [1, 2, 3, 5, 20, 1000], [0.0, 0.02, 0.05, 0.1, 0.3, 1e30]
    grew = 0
    for _ in range(5):
        d = _drafts(st, g, 12, r)
        d[d == 2] = 5
        n = np.zeros((len(betas), len(taus)), int)
        for i, be in enumerate(betas):
            for j, ta in enumerate(taus):
                st.reset()
                n[i, j] = st.verify_block_pp(0, d, be, ta)["n"]
        assert (np.diff(n, axis=0) >= 0).all() and (np.diff(n, axis=1) >= 0).all()
        grew += n[-1, -1] > n[0, 0]
    assert grew >= 3                                         # the relaxation does accept more on these blocks


@pytest.mark.parametrize("beta,tau", [(1, 0.0), (3, 0.05), (5, 0.3), (1000, 1e30)])
def test_loop_output_tokens_all_meet_the_rule(tiny, beta, tau):
    """Whatever the loop produced, token t is either the greedy choice given the output's own prefix or a token
    that meets the relaxed requirement given that prefix (scores re-derived by the cache-free full pass)."""
    m, st, g = tiny
    stream = synth.corrupt_stream(g[None, :], [len(g)], 0.6, synth.TINY.vocab, 3)[0]
    out, tr = st.gad_pp(None, 6, 24, beta, tau, override=stream)
    assert tr["n"].min() >= 1 and tr["n"].sum() == len(out)
    if beta == 1 and tau == 0.0:
        assert np.array_equal(out, g)
    mem = m.encode_memory(st.src)
    lg = m.decode_full(mem, np.concatenate([[0], out[:-1]]).astype(np.int32))
    relaxed = 0
    for t, tok in enumerate(out):
        top = int(np.argmax(lg[t]))
        if tok != top:
            relaxed += 1
            assert _brute(lg[t], int(tok), beta, tau)
            assert tok == stream[t]                         # only a drafted token can replace the greedy one
    if beta == 1000:
        assert relaxed > 0
        _, tr0 = st.gad_pp(None, 6, 24, 1, 0.0, override=stream)
        assert tr["iterations"] <= tr0["iterations"]

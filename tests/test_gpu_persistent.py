"""The persistent form of the decoder pass (decoder stack + projection as one kernel, selected with AD_MEGA=1):
same parity bars against the CPU checker as the default kernel chain, and the same ids as the chain."""
import numpy as np
import pytest

from oracle import ad_oracle as O
from paper_2205_10350_b200 import binding, synth
from tests import parity_util as P

pytestmark = pytest.mark.gpu
TOL_BF16 = 5e-2


@pytest.fixture()
def persistent(monkeypatch):
    monkeypatch.setenv("AD_MEGA", "1")          # read when a handle is created
    monkeypatch.setenv("AD_MEGA_TIMELINE", "1")


def _greedy_streams(om, src, lens, max_len, agreement, seed, vocab):
    B = len(lens)
    greedy = [om.state(src[b, : lens[b]]).greedy(int(max_len[b])) for b in range(B)]
    g = np.full((B, int(max(max_len))), synth.PAD, np.int32)
    gl = np.zeros(B, np.int32)
    for b in range(B):
        g[b, : len(greedy[b][0])] = greedy[b][0]
        gl[b] = len(greedy[b][0])
    return greedy, synth.corrupt_stream(g, gl, agreement, vocab, seed)


def test_mini_model_lockstep_generate_and_drafter(persistent):
    """Cluster size 4 (d_model 256), four ragged rows in one pass, drafter pass through the same kernel (gathered
    mask rows feed the projection)."""
    shape = synth.MINI_BF16
    w, wn = synth.make_weights(shape, 0), synth.make_weights(shape, 1)
    dec = binding.AggressiveDecoder(shape, w, wn, max_batch=4, max_src=20, max_tgt=15, kmax=15)   # drafter pass: 4 x 16 = 64 rows
    om, on = O.Model(shape, w, max_pos=32), O.Model(shape, wn, max_pos=32)
    wl = synth.Workload(9, shape, "IAD", 4, 1, 9, 20, 0, 15, 0.8, True)
    src, lens = synth.make_sources(wl)
    max_len = np.minimum(lens, 15)
    greedy, streams = _greedy_streams(om, src, lens, max_len, 0.8, 9, shape.vocab)
    tot = P.lockstep(dec, om, src, lens, list(streams), 15, max_len, TOL_BF16)
    assert tot["tokens"] == int(sum(len(x[0]) for x in greedy))
    tl = dec.debug_stage_timeline()
    assert (tl[:, 1] > tl[:, 0]).all() and (np.diff(tl[:, 0]) > 0).all(), "the persistent kernel did not run"
    print(f"mini, persistent pass: {tot}")
    for graph in (False, True):
        outs, _ = dec.generate(src, lens, mode="IAD", k=15, max_len=max_len, draft_override=streams, use_graph=graph)
        for b in range(4):
            P.check_free_run(outs[b], greedy[b][0], greedy[b][1], f"row {b}")
    outs, _ = dec.generate(src, lens, mode="GAD", k=6, max_len=max_len, run_drafter=True)
    for b in range(4):
        P.check_free_run(outs[b], greedy[b][0], greedy[b][1], f"GAD row {b}")
    r = np.random.default_rng(12)
    st = P.drafter_at_prefix(dec, on, src, lens, [r.integers(4, shape.vocab, size=n) for n in (3, 7, 0, 9)], 6, TOL_BF16)
    print(f"mini, persistent drafter pass at prefixes 3/7/0/9: {st}")
    dec.close()


def test_base_model_sentence_lockstep_and_same_ids_as_the_chain(persistent, monkeypatch):
    """Transformer-base, batch 1 (cluster size 8, 250 projection tiles): one sentence of the GEC-shaped workload in
    lock-step with the checker; then the same blocks through the default kernel chain give the same ids wherever the
    checker's margin is clear."""
    wl = synth.WORKLOADS[2]
    w = synth.make_weights(synth.BASE, 0)
    om = O.Model(synth.BASE, w, max_pos=64)
    src, lens = synth.make_sources(wl, 1)
    max_len = synth.max_out_lens(wl, lens)
    greedy, streams = _greedy_streams(om, src, lens, max_len, wl.agreement, wl.index, wl.shape.vocab)
    dec = binding.AggressiveDecoder(synth.BASE, w, max_batch=1, max_src=40, max_tgt=40, kmax=40)
    tot = P.lockstep(dec, om, src, lens, list(streams), 40, max_len, TOL_BF16)
    assert tot["tokens"] == len(greedy[0][0])
    print(f"base, persistent pass: {tot}")
    k = int(max_len[0])
    dec.encode(src, lens)
    ids_p, n_p = dec.verify_block(streams[:, :k], [k])
    lg_p = dec.debug_logits(k)
    dec.close()
    monkeypatch.setenv("AD_MEGA", "0")
    chain = binding.AggressiveDecoder(synth.BASE, w, max_batch=1, max_src=40, max_tgt=40, kmax=40)
    chain.encode(src, lens)
    ids_c, n_c = chain.verify_block(streams[:, :k], [k])
    lg_c = chain.debug_logits(k)
    assert np.abs(lg_p - lg_c).max() < TOL_BF16
    res = om.state(src[0, : lens[0]]).verify_block(0, streams[0, :k])
    clear = res["margin"] > P.MARGIN
    assert np.array_equal(ids_p[0, :k][clear], ids_c[0, :k][clear])
    chain.close()


def test_big_model_block_and_bart_sized_ragged_projection(persistent):
    """d_model 1024 (two K blocks per CTA, two projection jobs per cluster in the wide stages) and the BART-base-sized
    shape (cluster size 4, vocabulary 50265: ragged last projection tile)."""
    for shape, k in ((synth.BIG, 25), (synth.BART_BASE_SIZED, 10)):
        w = synth.make_weights(shape, 0)
        dec = binding.AggressiveDecoder(shape, w, max_batch=1, max_src=24, max_tgt=32, kmax=k)
        om = O.Model(shape, w, max_pos=40)
        r = np.random.default_rng(31)
        src = r.integers(4, shape.vocab, size=(1, 24)).astype(np.int32)
        lens = np.array([24], np.int32)
        g, _ = om.state(src[0]).greedy(2 * k)
        stream = synth.corrupt_stream(g[None, :], [len(g)], 0.8, shape.vocab, 31)[0]
        tot = P.lockstep(dec, om, src, lens, [stream], k, [len(g)], TOL_BF16, max_steps=2)
        assert tot["steps"] == 2 and tot["worst_logit_err"] < TOL_BF16
        tl = dec.debug_stage_timeline()
        assert (tl[:, 1] > tl[:, 0]).all()
        print(f"{shape.name}, persistent pass: {tot}")
        dec.close()

"""Parity of the CUDA path with the CPU checker on the five workload recipes, through the C ABI.

Bars: token ids, accepted lengths and cache lengths exact wherever the checker's top-1/top-2 score gap
exceeds 0.1; scores within 1e-3 (FP32 model) / 5e-2 (BF16 models) max-abs.
"""
import numpy as np
import pytest

from oracle import ad_oracle as O
from paper_2205_10350_b200 import binding, synth
from tests import parity_util as P

pytestmark = pytest.mark.gpu
TOL_FP32, TOL_BF16 = 1e-3, 5e-2


def make(shape, wl_batch, max_src, max_tgt, kmax, drafter=False, std=0.02):
    w = synth.make_weights(shape, 0, std=std)
    wn = synth.make_weights(shape, 1, std=std) if drafter else None
    dec = binding.AggressiveDecoder(shape, w, wn, max_batch=wl_batch, max_src=max_src, max_tgt=max_tgt, kmax=kmax)
    om = O.Model(shape, w, max_pos=max(max_src, max_tgt + 1))
    on = O.Model(shape, wn, max_pos=max(max_src, max_tgt + 1)) if drafter else None
    return dec, om, on


# ------------------------------------------------------------------------------------------ workload 1
@pytest.fixture(scope="module")
def tiny():
    return make(synth.TINY, 1, 16, 24, 17, drafter=True)


def test_tiny_encoder_memory(tiny):
    dec, om, _ = tiny
    src, lens = synth.make_sources(synth.WORKLOADS[1])
    dec.encode(src, lens)
    mem = dec.debug_encoder_memory(0, int(lens[0]))
    assert np.abs(mem - om.state(src[0, :lens[0]]).memory()).max() < 1e-4


def test_tiny_lockstep_source_copy_drafts(tiny):
    dec, om, _ = tiny
    src, lens = synth.make_sources(synth.WORKLOADS[1])
    stream = np.concatenate([src[0, :16], np.full(16, -1, np.int32)])
    tot = P.lockstep(dec, om, src, lens, [stream], 17, [24], TOL_FP32)
    assert tot["tokens"] == 24 and tot["worst_logit_err"] < TOL_FP32


def test_tiny_input_guided_generate_is_identical_to_greedy(tiny):
    dec, om, _ = tiny
    src, lens = synth.make_sources(synth.WORKLOADS[1])
    st = om.state(src[0, :lens[0]])
    g, margin = st.greedy(24)
    ref_out, ref_tr = st.iad(17, 24)
    for graph in (False, True):
        outs, stats = dec.generate(src, lens, mode="IAD", k=17, max_len=[24], use_graph=graph)
        assert np.array_equal(outs[0], g)
        assert stats["iterations"] == ref_tr["iterations"] and stats["offered"] == ref_tr["offered"]
        assert stats["accepted"] == len(g)
    outs, stats = dec.generate(src, lens, mode="IAD", k=1, max_len=[24])      # k = 1 is greedy decoding
    assert np.array_equal(outs[0], g) and stats["iterations"] == len(g)


def test_tiny_generalized_mode_with_real_drafter(tiny):
    dec, om, on = tiny
    src, lens = synth.make_sources(synth.WORKLOADS[1])
    st = om.state(src[0, :lens[0]])
    g, _ = st.greedy(24)
    ref_out, ref_tr = st.gad(on, 5, 24)
    outs, stats = dec.generate(src, lens, mode="GAD", k=5, max_len=[24], run_drafter=True)
    assert np.array_equal(outs[0], g)
    assert stats["iterations"] == ref_tr["iterations"]
    # drafter block alone, at the start of decoding
    dec.encode(src, lens)
    d, k = dec.draft_block(5)
    ref_d, ref_m = on.nar_draft(on.encode_memory(src[0, :lens[0]]), [0], 5)
    assert k[0] == 5
    for i in range(5):
        assert d[0, i] == ref_d[i] or ref_m[i] <= P.MARGIN


def test_tiny_drafter_block_at_nonempty_prefix(tiny):
    """Section 3.2.1: the drafter conditions on the accepted prefix.  FP32 model: ids identical to the checker's."""
    dec, _, on = tiny
    src, lens = synth.make_sources(synth.WORKLOADS[1])
    r = np.random.default_rng(3)
    for j, k in ((1, 5), (7, 17), (19, 9), (23, 4)):      # the last two are clipped by the remaining length
        prefix = r.integers(4, synth.TINY.vocab, size=j)
        st = P.drafter_at_prefix(dec, on, src, lens, [prefix], k, TOL_FP32, exact=True)
        print(f"tiny drafter j={j} k={k}: {st}")


def test_varied_fp32_drafter_ragged_prefixes():
    """Three rows with different prefix lengths (one empty) through one drafter pass; larger weights so that the
    prefix really changes the drafts."""
    shape = synth.ModelShape("vary", 64, 2, 128, 40, 1, 2, "fp32")
    dec, om, on = make(shape, 3, 12, 30, 13, drafter=True, std=0.15)
    r = np.random.default_rng(6)
    lens = np.array([12, 7, 9], np.int32)
    src = np.full((3, 12), synth.PAD, np.int32)
    for b in range(3):
        src[b, : lens[b]] = r.integers(4, 40, size=lens[b])
    prefixes = [r.integers(4, 40, size=n) for n in (14, 0, 5)]
    st = P.drafter_at_prefix(dec, on, src, lens, prefixes, 6, TOL_FP32, exact=True)
    print(f"varied drafter: {st}")
    # the prefix matters: the same rows at an empty prefix draft something else somewhere
    d0 = on.nar_draft(on.encode_memory(src[0, :12]), [0], 6)[0]
    d1 = on.nar_draft(on.encode_memory(src[0, :12]), [0] + [int(t) for t in prefixes[0]], 6)[0]
    assert not np.array_equal(d0, d1)
    dec.close()


# A model with larger weights decodes to varied text, which exercises suffix matching, rollback and EOS.
@pytest.mark.parametrize("seed_std", [0.08, 0.15])
def test_varied_fp32_model_all_modes(seed_std):
    shape = synth.ModelShape("vary", 64, 2, 128, 40, 1, 2, "fp32")
    dec, om, on = make(shape, 3, 12, 30, 13, drafter=True, std=seed_std)
    r = np.random.default_rng(5)
    lens = np.array([12, 7, 9], np.int32)
    src = np.full((3, 12), synth.PAD, np.int32)
    for b in range(3):
        src[b, : lens[b]] = r.integers(4, 40, size=lens[b])
    max_len = np.array([30, 18, 25], np.int32)
    greedy = [om.state(src[b, : lens[b]]).greedy(int(max_len[b])) for b in range(3)]
    outs, stats = dec.generate(src, lens, mode="IAD", k=13, max_len=max_len)
    iters = 0
    for b in range(3):
        assert P.check_free_run(outs[b], greedy[b][0], greedy[b][1], f"IAD row {b}") is None
        iters += om.state(src[b, : lens[b]]).iad(13, int(max_len[b]))[1]["iterations"]
    assert stats["row_iterations"] == iters
    outs, _ = dec.generate(src, lens, mode="GAD", k=4, max_len=max_len, run_drafter=True)
    for b in range(3):
        assert P.check_free_run(outs[b], greedy[b][0], greedy[b][1], f"GAD row {b}") is None
    streams = np.full((3, 30), 5, np.int32)
    for b in range(3):
        g = greedy[b][0]
        streams[b, : len(g)] = np.where(r.random(len(g)) < 0.7, g, 6)
    outs, stats = dec.generate(src, lens, mode="GAD", k=6, max_len=max_len, draft_override=streams)
    for b in range(3):
        assert P.check_free_run(outs[b], greedy[b][0], greedy[b][1], f"stream row {b}") is None
    tot = P.lockstep(dec, om, src, lens, list(streams), 6, max_len, TOL_FP32)
    assert tot["flipped"] == 0


# ------------------------------------------------------------------------------------------ small BF16
def test_mini_bf16_lockstep_and_generate():
    shape = synth.MINI_BF16
    dec, om, on = make(shape, 4, 20, 24, 16, drafter=True)
    wl = synth.Workload(9, shape, "IAD", 4, 1, 9, 20, 0, 16, 0.8, True)
    src, lens = synth.make_sources(wl)
    max_len = np.minimum(lens, 24)
    greedy = [om.state(src[b, : lens[b]]).greedy(int(max_len[b])) for b in range(4)]
    g = np.full((4, 24), synth.PAD, np.int32)
    for b in range(4):
        g[b, : len(greedy[b][0])] = greedy[b][0]
    streams = synth.corrupt_stream(g, max_len, 0.8, shape.vocab, 9)
    tot = P.lockstep(dec, om, src, lens, list(streams), 16, max_len, TOL_BF16)
    assert tot["tokens"] == int(sum(len(x[0]) for x in greedy))
    outs, _ = dec.generate(src, lens, mode="IAD", k=16, max_len=max_len, draft_override=streams)
    for b in range(4):
        P.check_free_run(outs[b], greedy[b][0], greedy[b][1], f"row {b}")
    outs, _ = dec.generate(src, lens, mode="GAD", k=8, max_len=max_len, run_drafter=True)
    for b in range(4):
        P.check_free_run(outs[b], greedy[b][0], greedy[b][1], f"GAD row {b}")
    # drafter at ragged non-empty prefixes (Section 3.2.1)
    r = np.random.default_rng(12)
    prefixes = [r.integers(4, shape.vocab, size=n) for n in (3, 11, 0, 17)]
    st = P.drafter_at_prefix(dec, on, src, lens, prefixes, 8, TOL_BF16)
    print(f"mini bf16 drafter at prefixes 3/11/0/17: {st}")


def test_mini_bf16_long_targets_reach_the_key_parallel_attention():
    """Targets of up to 300 tokens: self-attention rows hold hundreds of keys, so the verifier's block-causal attention
    (per-token key counts) and the drafter's bidirectional attention over prefix + masks run in the kernel that spreads a
    row's keys over the warps of a CTA (1, 2 and 4 query tiles per CTA; ragged rows of 270 and 130 committed tokens).
    The verifier's block is compared with the checker's plain forward over the whole sequence (no cache)."""
    shape = synth.MINI_BF16
    dec, om, on = make(shape, 2, 20, 300, 20, drafter=True)
    r = np.random.default_rng(31)
    src = r.integers(4, shape.vocab, size=(2, 20)).astype(np.int32)
    lens = np.array([20, 13], np.int32)
    prefixes = [r.integers(4, shape.vocab, size=n).astype(np.int32) for n in (270, 130)]
    st = P.drafter_at_prefix(dec, on, src, lens, prefixes, 20, TOL_BF16)
    print(f"mini bf16 drafter at prefixes 270/130: {st}")
    ks = [20, 9]
    drafts = np.full((2, 20), -1, np.int32)
    for b in range(2):
        drafts[b, : ks[b]] = r.integers(4, shape.vocab, size=ks[b])
    ids, n = dec.verify_block(drafts, ks)
    lg = dec.debug_logits(sum(ks))
    off, exact = 0, 0
    for b in range(2):
        k, j = ks[b], len(prefixes[b])
        mem = om.encode_memory(src[b, : lens[b]])
        seq = np.concatenate([[om.bos], prefixes[b], drafts[b, : k - 1]]).astype(np.int32)
        ref = om.decode_full(mem, seq, causal=True)[j: j + k]
        assert np.abs(lg[off: off + k] - ref).max() <= TOL_BF16
        for i in range(k):
            top = np.argsort(-ref[i], kind="stable")[:2]
            if ref[i][top[0]] - ref[i][top[1]] > P.MARGIN:
                assert ids[b, i] == top[0], (b, i)
                exact += 1
            else:
                assert ids[b, i] in top
        n_self, _ = P.OPS.accept(ids[b, :k], drafts[b, :k], eos=2)
        assert n[b] == n_self
        off += k
    assert exact >= 5
    dec.close()


# ------------------------------------------------------------------------------------------ workloads 2, 3
@pytest.fixture(scope="module")
def base_weights():
    return synth.make_weights(synth.BASE, 0)


def _greedy_streams(om, src, lens, max_len, agreement, wl_index, vocab):
    B = len(lens)
    greedy = [om.state(src[b, : lens[b]]).greedy(int(max_len[b])) for b in range(B)]
    g = np.full((B, int(max(max_len))), synth.PAD, np.int32)
    gl = np.zeros(B, np.int32)
    for b in range(B):
        g[b, : len(greedy[b][0])] = greedy[b][0]
        gl[b] = len(greedy[b][0])
    return greedy, synth.corrupt_stream(g, gl, agreement, vocab, wl_index)


def test_workload2_base_batch1(base_weights):
    wl = synth.WORKLOADS[2]
    dec = binding.AggressiveDecoder(synth.BASE, base_weights, max_batch=1, max_src=40, max_tgt=40, kmax=40)
    om = O.Model(synth.BASE, base_weights, max_pos=64)
    for sent in range(3):
        src, lens = synth.make_sources(wl, sent)
        max_len = synth.max_out_lens(wl, lens)
        greedy, streams = _greedy_streams(om, src, lens, max_len, wl.agreement, wl.index, wl.shape.vocab)
        kcap = min(wl.k, dec.kmax)       # outputs are at most 40 tokens here, so the cap of 64 never binds
        tot = P.lockstep(dec, om, src, lens, list(streams), kcap, max_len, TOL_BF16)
        assert tot["tokens"] == len(greedy[0][0])
        outs, stats = dec.generate(src, lens, mode="IAD", k=kcap, max_len=max_len, draft_override=streams)
        P.check_free_run(outs[0], greedy[0][0], greedy[0][1], f"sentence {sent}")
        assert 1 <= stats["iterations"] <= len(outs[0])


def test_workload3_base_batch32(base_weights):
    wl = synth.WORKLOADS[3]
    dec = binding.AggressiveDecoder(synth.BASE, base_weights, max_batch=32, max_src=64, max_tgt=64, kmax=64)
    om = O.Model(synth.BASE, base_weights, max_pos=80)
    src, lens = synth.make_sources(wl)
    max_len = synth.max_out_lens(wl, lens)
    greedy, streams = _greedy_streams(om, src, lens, max_len, wl.agreement, wl.index, wl.shape.vocab)
    tot = P.lockstep(dec, om, src, lens, list(streams), wl.k, max_len, TOL_BF16, max_steps=2)
    assert tot["steps"] == 2
    print(f"recipe 3, two iterations, all 32 rows: {tot}")
    # four rows to the END of their sentences in lock-step with the checker while all 32 rows run (the other 28 follow the
    # library's own trajectory): per-row accepted lengths and cache commits stay independent in a wide ragged batch
    tot = P.lockstep(dec, om, src, lens, list(streams), wl.k, max_len, TOL_BF16, check_rows=[0, 5, 17, 31])
    assert tot["tokens"] == sum(len(greedy[b][0]) for b in (0, 5, 17, 31))
    print(f"recipe 3, rows 0/5/17/31 to completion: {tot}")
    outs, stats = dec.generate(src, lens, mode="IAD", k=wl.k, max_len=max_len, draft_override=streams)
    for b in range(wl.batch):
        P.check_free_run(outs[b], greedy[b][0], greedy[b][1], f"row {b}")
    ln, _, fin = dec.state()
    assert (fin == 1).all() and all(ln[b] == len(outs[b]) for b in range(wl.batch))


# ------------------------------------------------------------------------------------------ workloads 4, 5
def _drafter_parity(dec, on, src, lens, k):
    """Drafter block at the start of decoding against the checker's drafter forward."""
    d, kk = dec.draft_block(k)
    for b in range(len(lens)):
        ref_d, ref_m = on.nar_draft(on.encode_memory(src[b, : lens[b]]), [0], k)
        assert kk[b] == k
        for i in range(k):
            assert d[b, i] == ref_d[i] or ref_m[i] <= P.MARGIN, (b, i, d[b, i], ref_d[i], ref_m[i])


def test_workload4_big_generalized():
    wl = synth.WORKLOADS[4]
    dec, om, on = make(synth.BIG, 1, 50, 50, 25, drafter=True)
    src, lens = synth.make_sources(wl, 0)
    max_len = synth.max_out_lens(wl, lens)
    greedy, streams = _greedy_streams(om, src, lens, max_len, wl.agreement, wl.index, wl.shape.vocab)
    dec.encode(src, lens)
    _drafter_parity(dec, on, src, lens, wl.k)
    st = P.drafter_at_prefix(dec, on, src, lens, [greedy[0][0][:9]], wl.k, TOL_BF16)
    print(f"big drafter at a 9-token prefix: {st}")
    tot = P.lockstep(dec, om, src, lens, list(streams), wl.k, max_len, TOL_BF16)     # the whole sentence
    assert tot["tokens"] == len(greedy[0][0])
    print(f"recipe 4, one sentence to completion: {tot}")
    outs, stats = dec.generate(src, lens, mode="GAD", k=wl.k, max_len=max_len, draft_override=streams, run_drafter=True)
    P.check_free_run(outs[0], greedy[0][0], greedy[0][1], "big")


def test_big_model_batch_of_four():
    """Transformer-big, four rows, 32-token sources, blocks of 25: passes of 100 and 128 tokens, whose projections run
    K loops of several ring rounds (K = 1024 and 4096) on short rings shared by two CTAs per SM.  Rows 0 and 3 follow the
    checker for two iterations; the other rows share their passes."""
    shape = synth.BIG
    dec, om, _ = make(shape, 4, 32, 50, 25)
    r = np.random.default_rng(44)
    src = r.integers(4, shape.vocab, size=(4, 32)).astype(np.int32)
    lens = np.array([32, 20, 27, 32], np.int32)
    max_len = np.full(4, 50, np.int32)
    streams = [r.integers(4, shape.vocab, size=50).astype(np.int32) for _ in range(4)]
    tot = P.lockstep(dec, om, src, lens, streams, 25, max_len, TOL_BF16, max_steps=2, check_rows=[0, 3])
    print(f"big, batch 4, two iterations, rows 0 and 3: {tot}")
    assert tot["steps"] == 2
    dec.close()


def test_workload5_base_long_source_batch8(base_weights):
    wl = synth.WORKLOADS[5]
    wn = synth.make_weights(synth.BASE, 1)
    dec = binding.AggressiveDecoder(synth.BASE, base_weights, wn, max_batch=8, max_src=400, max_tgt=80, kmax=25)
    om = O.Model(synth.BASE, base_weights, max_pos=401)
    on = O.Model(synth.BASE, wn, max_pos=401)
    src, lens = synth.make_sources(wl)
    max_len = synth.max_out_lens(wl, lens)
    # All 8 rows in lock-step with the checker for 12 iterations at agreement 0.6 (about 2.5 tokens accepted per row and
    # iteration): every iteration rolls the rejected part of a 25-token block back, and the cache is some 25 positions
    # deep by the end.  The checker pays the 400-token encoder once per row.
    T = 40
    states = [om.state(src[b, : lens[b]], cap=80) for b in range(8)]
    dec.encode(src, lens)
    mem = dec.debug_encoder_memory(1, int(lens[1]))
    assert np.abs(mem - states[1].memory()).max() < TOL_BF16
    _drafter_parity(dec, on, src[:1], lens[:1], 5)
    gT = [st.greedy(T) for st in states]
    g = np.full((8, 80), synth.PAD, np.int32)
    gl = np.zeros(8, np.int32)
    for b in range(8):
        g[b, : len(gT[b][0])] = gT[b][0]; gl[b] = len(gT[b][0])
    streams = synth.corrupt_stream(g, gl, wl.agreement, wl.shape.vocab, wl.index)
    tot = P.lockstep(dec, om, src, lens, list(streams), wl.k, np.full(8, T), TOL_BF16, max_steps=12, states=states)
    assert tot["steps"] == 12 or tot["tokens"] == int(gl.sum())
    ln, _, _ = dec.state()
    print(f"recipe 5, 8 rows x {tot['steps']} iterations, cache depths {list(ln)}: {tot}")
    assert max(ln) >= 20
    # full batch, free running with the drafter: the loop must terminate and agree with the checker's greedy output
    outs, stats = dec.generate(src, lens, mode="GAD", k=wl.k, max_len=np.full(8, T, np.int32), draft_override=streams,
                               run_drafter=True)
    assert all(1 <= len(o) <= T for o in outs)
    for b in range(8):
        P.check_free_run(outs[b], gT[b][0], gT[b][1], f"row {b}")


def test_long_source_short_blocks(base_weights):
    """Few queries per row against hundreds of source keys: the attention variant in which the warps of a CTA
    split the keys of a row and merge their partial softmax results (blocks of at most 12 and of at most 30)."""
    r = np.random.default_rng(synth.MASTER_SEED + 77)
    B, S = 2, 300
    src = r.integers(4, synth.BASE.vocab, size=(B, S)).astype(np.int32)
    lens = np.array([S, 211], np.int32)
    src[1, 211:] = synth.PAD
    om = O.Model(synth.BASE, base_weights, max_pos=S + 1)
    states = [om.state(src[b, : lens[b]], cap=40) for b in range(B)]
    g = [st.greedy(10) for st in states]
    for kmax in (12, 30):
        dec = binding.AggressiveDecoder(synth.BASE, base_weights, max_batch=B, max_src=S, max_tgt=40, kmax=kmax)
        streams = np.full((B, 40), 11, np.int32)
        for b in range(B):
            streams[b, : len(g[b][0])] = g[b][0]
            streams[b, 6] = 13
        tot = P.lockstep(dec, om, src, lens, list(streams), kmax, [40, 40], TOL_BF16, max_steps=2)
        assert tot["steps"] == 2


# ------------------------------------------------------------------------------------------ other shapes
def test_deep_encoder_shallow_decoder_shape():
    """A 6-layer encoder over a 1-layer decoder (the layer split of the paper's 12+2 model, Section 4.1.2, at a width
    the checker finishes in seconds): input-guided lock-step run and free run."""
    shape = synth.ModelShape("deep_enc_mini", 256, 4, 512, 2048, 6, 1, "bf16")
    dec, om, _ = make(shape, 2, 18, 20, 19)
    wl = synth.Workload(10, shape, "IAD", 2, 1, 10, 18, 0, 19, 0.85, False)
    src, lens = synth.make_sources(wl)
    max_len = np.minimum(lens, 20)
    greedy = [om.state(src[b, : lens[b]]).greedy(int(max_len[b])) for b in range(2)]
    g = np.full((2, 20), synth.PAD, np.int32)
    for b in range(2):
        g[b, : len(greedy[b][0])] = greedy[b][0]
    streams = synth.corrupt_stream(g, max_len, 0.85, shape.vocab, 10)
    tot = P.lockstep(dec, om, src, lens, list(streams), 19, max_len, TOL_BF16)
    assert tot["tokens"] == int(sum(len(x[0]) for x in greedy))
    outs, _ = dec.generate(src, lens, mode="IAD", k=19, max_len=max_len)       # Algorithm 1 on the real sources
    for b in range(2):
        P.check_free_run(outs[b], greedy[b][0], greedy[b][1], f"row {b}")
    dec.close()


def test_twelve_plus_two_model_at_its_real_shape():
    """The 12-layer-encoder / 2-layer-decoder model of Section 4.1.2 at its real width (d_model 512, 8 heads, FFN 2048,
    vocabulary 32000): encoder memory after twelve layers, two lock-step verification steps and the free run."""
    shape = synth.DEEP_ENC
    dec, om, _ = make(shape, 1, 24, 24, 24)
    r = np.random.default_rng(41)
    src = r.integers(4, shape.vocab, size=(1, 24)).astype(np.int32)
    lens = np.array([20], np.int32)
    src[0, 20:] = synth.PAD
    st = om.state(src[0, :20])
    g, margin = st.greedy(20)
    stream = synth.corrupt_stream(g[None, :], [len(g)], 0.85, shape.vocab, 41)[0]
    dec.encode(src, lens)
    mem = dec.debug_encoder_memory(0, 20)
    assert np.abs(mem - st.memory()).max() < 5e-2
    tot = P.lockstep(dec, om, src, lens, [stream], 24, [20], TOL_BF16, max_steps=2)
    assert tot["steps"] == 2 and tot["worst_logit_err"] < TOL_BF16
    print(f"12+2 model: {tot}")
    outs, _ = dec.generate(src, lens, mode="IAD", k=24, max_len=[20], draft_override=stream[None, :])
    P.check_free_run(outs[0], g, margin, "12+2")
    dec.close()


def test_bart_base_sized_shape_two_steps():
    """d_model 768, 12 heads, FFN 3072, vocabulary 50265 (393 projection tiles, the last one ragged), the size of the
    models of Section 4.2.4: encoder memory and two lock-step verification steps of a 10-token block."""
    shape = synth.BART_BASE_SIZED
    dec, om, _ = make(shape, 1, 24, 24, 10)
    r = np.random.default_rng(31)
    src = r.integers(4, shape.vocab, size=(1, 24)).astype(np.int32)
    lens = np.array([24], np.int32)
    st = om.state(src[0])
    g, _ = st.greedy(20)
    stream = synth.corrupt_stream(g[None, :], [len(g)], 0.8, shape.vocab, 31)[0]
    dec.encode(src, lens)
    mem = dec.debug_encoder_memory(0, 24)
    assert np.abs(mem - st.memory()).max() < 5e-2
    tot = P.lockstep(dec, om, src, lens, [stream], 10, [20], TOL_BF16, max_steps=2)
    assert tot["steps"] == 2 and tot["worst_logit_err"] < TOL_BF16
    dec.close()

import numpy as np
import torch

from paper_2205_10350_b200 import synth


def test_bf16_rounding_matches_torch():
    a = np.random.default_rng(0).standard_normal(100000).astype(np.float32) * 0.02
    ref = torch.tensor(a).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(synth.round_to_bf16(a), ref)


def test_weights_are_seeded_and_bf16_exact():
    w1 = synth.make_weights(synth.MINI_BF16, 0)
    w2 = synth.make_weights(synth.MINI_BF16, 0)
    w3 = synth.make_weights(synth.MINI_BF16, 1)
    assert all(np.array_equal(w1[k], w2[k]) for k in w1)
    assert not np.array_equal(w1["emb"], w3["emb"])
    assert np.array_equal(synth.round_to_bf16(w1["emb"]), w1["emb"])
    assert abs(w1["emb"].std() - 0.02) < 0.002
    assert abs(w1["enc.0.ln1.g"].mean() - 1.0) < 0.01


def test_sources_follow_the_recipes():
    for idx, wl in synth.WORKLOADS.items():
        src, lens = synth.make_sources(wl)
        assert src.shape == (wl.batch, wl.src_len_hi)
        assert (lens >= wl.src_len_lo).all() and (lens <= wl.src_len_hi).all()
        for b in range(wl.batch):
            assert (src[b, : lens[b]] >= 4).all() and (src[b, : lens[b]] < wl.shape.vocab).all()
            assert (src[b, lens[b]:] == synth.PAD).all()


def test_corrupt_stream_rate_and_exclusion():
    g = np.random.default_rng(1).integers(4, 32000, size=(8, 5000)).astype(np.int32)
    c = synth.corrupt_stream(g, np.full(8, 5000), 0.9, 32000, 2)
    assert abs((c == g).mean() - 0.9) < 0.01
    assert (c >= 4).all() and (c < 32000).all()
    c2 = synth.corrupt_stream(g, np.full(8, 100), 0.0, 32000, 2)
    assert (c2[:, :100] != g[:, :100]).all() and np.array_equal(c2[:, 100:], g[:, 100:])

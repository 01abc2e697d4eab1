"""A property that holds at any size: a row's verified block does not depend on which other rows share its pass.

Batched passes of different sizes take different kernels and launch shapes (token tiles of 32, 64 or 128, split-K
factors, the attention kernel for few queries / many queries / hundreds of keys, the persistent projection kernel), a
single row takes the small-pass ones.  The scores of sampled rows of a ragged batch are compared with the same rows
verified alone; both sides are the library, so this pins no arithmetic -- the checker does that at sizes it can afford
(test_gpu_parity.py) -- but it ties every large-pass configuration to the small-pass path the checker follows
element by element.  Tolerance: the BF16 bar (the two sides differ in summation order only)."""
import numpy as np
import pytest

from paper_2205_10350_b200 import binding, synth

pytestmark = pytest.mark.gpu

CASES = [("base", synth.BASE, 8, 25, 400),       # 200-token capacity: 32-token tiles, keys spread over warps
         ("base", synth.BASE, 32, 30, 48),       # 960: 64-token tiles, tensor-core attention, persistent projection
         ("big", synth.BIG, 4, 25, 32),          # 100: K loops of several ring rounds
         ("big", synth.BIG, 16, 64, 32),         # 1024
         ("bart", synth.BART_BASE_SIZED, 6, 30, 40),   # 12 heads, K blocks not a power of two
         ("base", synth.BASE, 3, 64, 300)]       # 192: long sources with long blocks


@pytest.mark.parametrize("name,shape,B,k,S", CASES, ids=[f"{c[0]}-{c[2]}x{c[3]}-src{c[4]}" for c in CASES])
def test_batched_pass_agrees_with_single_row_passes(name, shape, B, k, S):
    r = np.random.default_rng(B * 1000 + k)
    w = synth.make_weights(shape, 0)
    src = r.integers(4, shape.vocab, size=(B, S)).astype(np.int32)
    lens = r.integers(max(1, S // 2), S + 1, size=B).astype(np.int32)
    ks = r.integers(1, k + 1, size=B).astype(np.int32)
    ks[B - 1] = k                                         # one full-length block
    drafts = r.integers(4, shape.vocab, size=(B, k)).astype(np.int32)
    dec = binding.AggressiveDecoder(shape, w, max_batch=B, max_src=S, max_tgt=k, kmax=k)
    dec.encode(src, lens)
    ids, n = dec.verify_block(drafts, ks)
    lg = dec.debug_logits(int(ks.sum()))
    dec.close()
    offs = np.concatenate([[0], np.cumsum(ks)])
    one = binding.AggressiveDecoder(shape, w, max_batch=1, max_src=S, max_tgt=k, kmax=k)
    worst = 0.0
    for b in sorted({0, B // 2, B - 1}):
        one.encode(src[b: b + 1], lens[b: b + 1])
        ids1, n1 = one.verify_block(drafts[b: b + 1], ks[b: b + 1])
        l1 = one.debug_logits(int(ks[b]))
        got = lg[offs[b]: offs[b + 1]]
        worst = max(worst, float(np.abs(got - l1).max()))
        # ids agree wherever the single-row scores leave no doubt
        top2 = np.sort(l1, axis=1)[:, -2:]
        clear = (top2[:, 1] - top2[:, 0]) > 0.1
        assert (ids[b, : ks[b]][clear] == ids1[0, : ks[b]][clear]).all()
    one.close()
    print(f"{name} B={B} k={k} S={S}: worst |batched - alone| = {worst:.4f}")
    assert worst <= 5e-2


DRAFT_CASES = [("base", synth.BASE, 8, 25, 400, 40), ("big", synth.BIG, 4, 25, 40, 30), ("mini", synth.MINI_BF16, 6, 16, 30, 200)]


@pytest.mark.parametrize("name,shape,B,k,S,T", DRAFT_CASES, ids=[f"{c[0]}-{c[2]}rows-prefix<={c[5]}" for c in DRAFT_CASES])
def test_batched_drafter_pass_agrees_with_single_row_passes(name, shape, B, k, S, T):
    """The same for the drafter's pass (Section 3.2.1): rows are walked to ragged prefixes by teacher forcing, then the
    draft scores of sampled rows of the batch are compared with the same rows drafted alone."""
    r = np.random.default_rng(B * 100 + T)
    w, wn = synth.make_weights(shape, 0), synth.make_weights(shape, 1)
    src = r.integers(4, shape.vocab, size=(B, S)).astype(np.int32)
    lens = r.integers(max(1, S // 2), S + 1, size=B).astype(np.int32)
    prefixes = [r.integers(4, shape.vocab, size=int(n)).astype(np.int32) for n in r.integers(0, T + 1, size=B)]

    def draft(dec, rows):
        dec.encode(src[rows], lens[rows])
        done = [0] * len(rows)
        while any(done[i] < len(prefixes[b]) for i, b in enumerate(rows)):
            ks = np.zeros(len(rows), np.int32)
            toks = np.full((len(rows), dec.kmax), -1, np.int32)
            for i, b in enumerate(rows):
                seg = prefixes[b][done[i]: done[i] + dec.kmax]
                ks[i] = len(seg)
                toks[i, : len(seg)] = seg
                done[i] += len(seg)
            dec.verify_block(toks, ks)
            dec.force_commit(toks, ks)
        d, kk = dec.draft_block(k)
        return d, kk, dec.debug_logits(int(kk.sum()), which=1)

    dec = binding.AggressiveDecoder(shape, w, wn, max_batch=B, max_src=S, max_tgt=T + k, kmax=k)
    d, kk, scores = draft(dec, list(range(B)))
    dec.close()
    offs = np.concatenate([[0], np.cumsum(kk)])
    one = binding.AggressiveDecoder(shape, w, wn, max_batch=1, max_src=S, max_tgt=T + k, kmax=k)
    worst = 0.0
    for b in sorted({0, B // 2, B - 1}):
        d1, k1, s1 = draft(one, [b])
        assert int(k1[0]) == int(kk[b])
        worst = max(worst, float(np.abs(scores[offs[b]: offs[b + 1]] - s1).max()))
    one.close()
    print(f"{name} B={B}: drafter worst |batched - alone| = {worst:.4f}")
    assert worst <= 5e-2


LOOP_CASES = [(5, 64, 40, "IAD", False), (8, 25, 100, "GAD", True), (32, 64, 48, "IAD", False), (4, 40, 300, "GAD", True)]


@pytest.mark.parametrize("B,k,S,mode,drafter", LOOP_CASES, ids=[f"{c[3]}-{c[0]}rows-k{c[1]}-src{c[2]}" for c in LOOP_CASES])
def test_decode_loop_as_one_graph_equals_direct_launches_at_every_pass_size(B, k, S, mode, drafter):
    """The whole loop (Algorithm 1 / Section 3.2) on the base model at several batch sizes: one graph launch with the
    device-side loop, the same call again, and direct launches with host polling must return identical tokens and
    iteration counts.  How many rows also equal the library's own greedy decoding (block size 1, other kernels and launch
    shapes) is printed: the method is lossless, so every row whose positions are all clear of near-ties does."""
    shape = synth.BASE
    r = np.random.default_rng(B * 7 + k)
    w = synth.make_weights(shape, 0)
    wn = synth.make_weights(shape, 1) if drafter else None
    T = max(48, k)
    dec = binding.AggressiveDecoder(shape, w, wn, max_batch=B, max_src=S, max_tgt=T, kmax=k)
    src = r.integers(4, shape.vocab, size=(B, S)).astype(np.int32)
    lens = r.integers(max(1, S // 2), S + 1, size=B).astype(np.int32)
    max_len = r.integers(8, T + 1, size=B).astype(np.int32)
    g, _ = dec.generate(src, lens, mode="IAD", k=1, max_len=max_len)
    gg = np.full((B, T), synth.PAD, np.int32)
    for b in range(B):
        gg[b, : len(g[b])] = g[b]
    kw = dict(mode=mode, k=k, max_len=max_len)
    if drafter:
        kw["run_drafter"] = True
    else:
        kw["draft_override"] = synth.corrupt_stream(gg, [len(x) for x in g], 0.8, shape.vocab, 3, B)
    a, sa = dec.generate(src, lens, use_graph=True, **kw)
    d, sd = dec.generate(src, lens, use_graph=False, **kw)
    c, sc = dec.generate(src, lens, use_graph=True, **kw)
    for b in range(B):
        assert np.array_equal(a[b], d[b]) and np.array_equal(a[b], c[b]), b
        assert 1 <= len(a[b]) <= max_len[b]
    assert sa["iterations"] == sd["iterations"] == sc["iterations"]
    same = sum(np.array_equal(a[b], g[b]) for b in range(B))
    print(f"B={B} k={k} S={S} {mode}: {sa['iterations']} iterations, {same}/{B} rows identical to block-size-1 decoding")
    assert same >= B - max(1, B // 4)          # near-ties may move a few rows off; a broken loop moves all of them
    dec.close()

"""Pins of the CPU checker's Transformer: library cross-check, positional table, cache identities."""
import numpy as np
import pytest
import torch

from oracle import ad_oracle as O
from paper_2205_10350_b200 import synth

SHAPE = synth.ModelShape("pin", 32, 4, 64, 50, 2, 2, "fp32")


@pytest.fixture(scope="module")
def weights():
    return synth.make_weights(SHAPE, 0, std=0.3)   # large std so every path matters numerically


def _torch_model(w, shape):
    """The same network assembled from torch.nn's own Transformer layers (post-LN, ReLU)."""
    d, H, F = shape.d_model, shape.n_heads, shape.d_ffn
    t = lambda a: torch.tensor(np.asarray(a, dtype=np.float64))

    def load_attn(mha, p):
        with torch.no_grad():
            mha.in_proj_weight.copy_(torch.cat([t(w[f"{p}.{n}.W"]).T for n in "qkv"], 0))
            mha.in_proj_bias.copy_(torch.cat([t(w[f"{p}.{n}.b"]) for n in "qkv"], 0))
            mha.out_proj.weight.copy_(t(w[f"{p}.o.W"]).T)
            mha.out_proj.bias.copy_(t(w[f"{p}.o.b"]))

    def load_lin(lin, p):
        with torch.no_grad():
            lin.weight.copy_(t(w[p + ".W"]).T)
            lin.bias.copy_(t(w[p + ".b"]))

    def load_ln(ln, p):
        with torch.no_grad():
            ln.weight.copy_(t(w[p + ".g"]))
            ln.bias.copy_(t(w[p + ".b"]))

    enc, dec = [], []
    for l in range(shape.n_enc):
        e = torch.nn.TransformerEncoderLayer(d, H, F, dropout=0.0, activation="relu", norm_first=False,
                                             layer_norm_eps=1e-5, dtype=torch.float64)
        load_attn(e.self_attn, f"enc.{l}.self"); load_ln(e.norm1, f"enc.{l}.ln1")
        load_lin(e.linear1, f"enc.{l}.ffn1"); load_lin(e.linear2, f"enc.{l}.ffn2"); load_ln(e.norm2, f"enc.{l}.ln2")
        enc.append(e.eval())
    for l in range(shape.n_dec):
        m = torch.nn.TransformerDecoderLayer(d, H, F, dropout=0.0, activation="relu", norm_first=False,
                                             layer_norm_eps=1e-5, dtype=torch.float64)
        load_attn(m.self_attn, f"dec.{l}.self"); load_ln(m.norm1, f"dec.{l}.ln1")
        load_attn(m.multihead_attn, f"dec.{l}.cross"); load_ln(m.norm2, f"dec.{l}.ln2")
        load_lin(m.linear1, f"dec.{l}.ffn1"); load_lin(m.linear2, f"dec.{l}.ffn2"); load_ln(m.norm3, f"dec.{l}.ln3")
        dec.append(m.eval())
    return enc, dec


def _pe(T, d):
    p = np.arange(T)[:, None]
    i = np.arange(0, d, 2)[None, :]
    ang = p / np.power(10000.0, i / d)
    out = np.zeros((T, d))
    out[:, 0::2] = np.sin(ang)
    out[:, 1::2] = np.cos(ang)
    return out


def test_positional_table_closed_form():
    m = O.Model(SHAPE, synth.make_weights(SHAPE, 0), max_pos=40, real="f64")
    pe = m.pe()
    assert np.array_equal(pe[0], np.tile([0.0, 1.0], SHAPE.d_model // 2))
    assert np.allclose(pe, _pe(40, SHAPE.d_model), atol=1e-14)
    # the first pair has wavelength 2*pi: PE(p, 0) = sin(p)
    assert np.allclose(pe[:, 0], np.sin(np.arange(40)), atol=1e-14)


@pytest.mark.parametrize("causal", [True, False])
def test_whole_model_matches_torch_nn_transformer(weights, causal):
    src = np.array([7, 9, 4, 33, 21, 8], np.int32)
    tok = np.array([0, 5, 11, 42, 6], np.int32)
    m = O.Model(SHAPE, weights, max_pos=32, real="f64")
    mem = m.encode_memory(src)
    logits = m.decode_full(mem, tok, causal=causal)

    enc, dec = _torch_model(weights, SHAPE)
    d = SHAPE.d_model
    emb = torch.tensor(weights["emb"].astype(np.float64))
    with torch.no_grad():
        x = (emb[torch.tensor(src, dtype=torch.long)] * np.sqrt(d) + torch.tensor(_pe(len(src), d))).unsqueeze(1)
        for e in enc:
            x = e(x)
        assert np.allclose(mem, x.squeeze(1).numpy(), atol=1e-9)
        y = (emb[torch.tensor(tok, dtype=torch.long)] * np.sqrt(d) + torch.tensor(_pe(len(tok), d))).unsqueeze(1)
        mask = torch.nn.Transformer.generate_square_subsequent_mask(len(tok), dtype=torch.float64) if causal else None
        for dl in dec:
            y = dl(y, x, tgt_mask=mask)
        ref = (y.squeeze(1) @ emb.T).numpy()
    assert np.allclose(logits, ref, atol=1e-8)


def test_f32_checker_close_to_f64_checker(weights):
    src = np.array([7, 9, 4, 33, 21, 8], np.int32)
    tok = np.array([0, 5, 11, 42, 6], np.int32)
    a = O.Model(SHAPE, weights, max_pos=32, real="f32")
    b = O.Model(SHAPE, weights, max_pos=32, real="f64")
    la = a.decode_full(a.encode_memory(src), tok)
    lb = b.decode_full(b.encode_memory(src), tok)
    assert np.abs(la - lb).max() < 5e-4 * max(1.0, np.abs(lb).max())


@pytest.mark.parametrize("real", ["f32", "f64"])
def test_incremental_cache_equals_full_recompute_bit_for_bit(weights, real):
    src = np.array([7, 9, 4, 33, 21, 8, 12], np.int32)
    tok = np.array([0, 5, 11, 42, 6, 17, 23, 9], np.int32)
    m = O.Model(SHAPE, weights, max_pos=32, real=real)
    full = m.decode_full(m.encode_memory(src), tok, causal=True)
    # (a) one block; (b) three blocks with commits; (c) single steps  -- Eq. (1): same scores
    st = m.state(src)
    assert np.array_equal(st.decode_block(tok), full)
    st.reset()
    got = []
    for a, b in ((0, 3), (3, 4), (4, 8)):
        got.append(st.decode_block(tok[a:b]))
        st.commit(b - a)
    assert np.array_equal(np.concatenate(got), full)
    st.reset()
    got = []
    for t in tok:
        got.append(st.decode_block([t]))
        st.commit(1)
    assert np.array_equal(np.concatenate(got), full)


def test_rollback_discards_rejected_positions(weights):
    """Positions written by a rejected part of a block must not influence later calls."""
    src = np.array([7, 9, 4, 33], np.int32)
    m = O.Model(SHAPE, weights, max_pos=32, real="f32")
    st = m.state(src)
    st.decode_block([0, 5, 11, 42, 6])     # tentative K/V for 5 positions
    st.commit(2)                           # keep two of them
    after = st.decode_block([30, 31])
    ref = m.decode_full(m.encode_memory(src), np.array([0, 5, 30, 31], np.int32))[2:]
    assert np.array_equal(after, ref)
    st.commit(2)
    st.commit(-3)                          # negative commit = roll the length back
    assert st.len == 1
    again = st.decode_block([5, 30])
    ref2 = m.decode_full(m.encode_memory(src), np.array([0, 5, 30], np.int32))[1:]
    assert np.array_equal(again, ref2)


def test_zero_sublayers_make_the_choice_depend_on_the_last_token_only():
    """With every projection and FFN matrix zero each sublayer adds a constant bias, so the decoder
    output at a position depends only on that position's own embedding: greedy decoding can be
    enumerated token by token."""
    w = synth.make_weights(SHAPE, 0, std=0.3)
    for k in w:
        if k.endswith(".W"):
            w[k] = np.zeros_like(w[k])
    m = O.Model(SHAPE, w, max_pos=32, real="f64")
    src = np.array([5, 6, 7], np.int32)
    st = m.state(src)
    a = st.decode_block([0, 9, 9, 13])
    # positions 1 and 2 hold the same token but different positions -> differ only through PE;
    # a one-token call at position 0 with the same token as a later call at position 0 is identical
    st2 = m.state(np.array([40, 41, 42, 43, 44], np.int32))   # other source: must not matter
    b = st2.decode_block([0, 9, 9, 13])
    assert np.allclose(a, b, atol=1e-12)


# ---------------------------------------------------------------------------------------------------
# Pins of the drafter forward (Section 3.2 "Draft", Section 3.2.1): inputs (o_0..o_j, k x [MASK]) at positions
# 0..j+k, bidirectional attention, drafts = greedy choices at the k mask positions.
# ---------------------------------------------------------------------------------------------------
def _ln(x, g, b, eps=1e-5):
    mu = x.mean()
    var = ((x - mu) ** 2).mean()
    return (x - mu) / np.sqrt(var + eps) * g + b


def _zero_sublayer_choice(w, shape, token, pos):
    """Closed form of the decoder's greedy choice for one (token, position) when every projection and FFN matrix
    is zero: each sublayer adds only its output bias to the residual before its LayerNorm."""
    d = shape.d_model
    x = np.asarray(w["emb"], np.float64)[token] * np.sqrt(d) + _pe(pos + 1, d)[pos]
    for l in range(shape.n_dec):
        p = f"dec.{l}"
        x = _ln(x + w[f"{p}.self.o.b"], w[f"{p}.ln1.g"], w[f"{p}.ln1.b"])
        x = _ln(x + w[f"{p}.cross.o.b"], w[f"{p}.ln2.g"], w[f"{p}.ln2.b"])
        x = _ln(x + w[f"{p}.ffn2.b"], w[f"{p}.ln3.g"], w[f"{p}.ln3.b"])
    logits = np.asarray(w["emb"], np.float64) @ x
    order = np.argsort(-logits, kind="stable")
    return int(order[0]), float(logits[order[0]] - logits[order[1]])


def test_drafter_block_on_a_zero_sublayer_model_has_a_closed_form():
    """With all matrices zero the drafter's choice at mask slot t is a function of ([MASK], position j+1+t) alone, which
    is evaluated here directly; a drafter that fed [PAD], read the rows one off, or numbered the positions from the
    block start instead of from 0 gives another id or another top-1/top-2 gap (checked below by evaluating those wrong
    forms)."""
    w = synth.make_weights(SHAPE, 3, std=0.3)
    for name in w:
        if name.endswith(".W"):
            w[name] = np.zeros_like(w[name])
    m = O.Model(SHAPE, w, max_pos=40, real="f64")
    mem = m.encode_memory(np.array([5, 6, 7, 8], np.int32))
    differs_pad = differs_shift = differs_origin = 0
    for j, k in ((0, 5), (3, 4), (7, 9), (12, 1)):
        prefix = [0] + [int(t) for t in np.random.default_rng(j).integers(4, SHAPE.vocab, size=j)]
        draft, margin = m.nar_draft(mem, prefix, k)
        for t in range(k):
            want, gap = _zero_sublayer_choice(w, SHAPE, m.mask, j + 1 + t)
            assert draft[t] == want, (j, k, t)
            assert abs(margin[t] - gap) < 1e-9
            other = lambda r: r[0] != want or abs(r[1] - gap) > 1e-6     # another id, or another top-1/top-2 gap
            differs_pad += other(_zero_sublayer_choice(w, SHAPE, m.pad, j + 1 + t))
            differs_shift += other(_zero_sublayer_choice(w, SHAPE, m.mask, j + t))
            differs_origin += other(_zero_sublayer_choice(w, SHAPE, m.mask, t)) if j > 0 else 1
    # the pin has teeth: each plausible mistake changes every one of the 19 (id, gap) pairs
    assert differs_pad == 19 and differs_shift == 19 and differs_origin == 19


@pytest.mark.parametrize("j,k", [(0, 4), (2, 3), (5, 6)])
def test_drafter_block_matches_torch_nn_transformer_without_a_mask(weights, j, k):
    """The full drafter forward (non-zero weights) against torch.nn's decoder layers run without a target mask over
    (prefix, k x [MASK]): same ids at rows j+1 .. j+k, same top-1/top-2 gaps; and a causal run disagrees, so the
    bidirectional attention is really exercised."""
    src = np.array([7, 9, 4, 33, 21, 8], np.int32)
    m = O.Model(SHAPE, weights, max_pos=32, real="f64")
    mem = m.encode_memory(src)
    prefix = [0] + [int(t) for t in np.random.default_rng(100 + j).integers(4, SHAPE.vocab, size=j)]
    draft, margin = m.nar_draft(mem, prefix, k)

    enc, dec = _torch_model(weights, SHAPE)
    d = SHAPE.d_model
    emb = torch.tensor(weights["emb"].astype(np.float64))
    tok = np.array(prefix + [m.mask] * k)
    with torch.no_grad():
        x = (emb[torch.tensor(src, dtype=torch.long)] * np.sqrt(d) + torch.tensor(_pe(len(src), d))).unsqueeze(1)
        for e in enc:
            x = e(x)
        outs = {}
        for causal in (False, True):
            y = (emb[torch.tensor(tok, dtype=torch.long)] * np.sqrt(d) + torch.tensor(_pe(len(tok), d))).unsqueeze(1)
            mask = torch.nn.Transformer.generate_square_subsequent_mask(len(tok), dtype=torch.float64) if causal else None
            for dl in dec:
                y = dl(y, x, tgt_mask=mask)
            outs[causal] = (y.squeeze(1) @ emb.T).numpy()
    ref = outs[False][j + 1:]
    assert np.array_equal(draft, ref.argmax(1))
    top2 = np.sort(ref, axis=1)[:, -2:]
    assert np.allclose(margin, top2[:, 1] - top2[:, 0], atol=1e-8)
    if k > 1:      # earlier mask slots see later ones only when attention is bidirectional
        assert np.abs(outs[True][j + 1:-1] - ref[:-1]).max() > 1e-6

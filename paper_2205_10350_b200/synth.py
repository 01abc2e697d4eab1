"""Seeded synthetic inputs: model shapes, weights, sources and corrupted draft streams.

This module holds no arithmetic of the decoding method.  It only draws random
numbers and lays them out under names; both the CUDA path and the CPU checker
read their inputs from here and pack them into their own layouts themselves.

Weight convention of the returned dict: a projection named ``*.W`` has shape
``[in_features, out_features]`` (``y = x @ W + b``); ``emb`` is ``[vocab, d_model]``.
All arrays are float32.  For ``dtype == "bf16"`` every value has been rounded once
(round-to-nearest-even) to a bfloat16-representable float32, so a consumer may
narrow it to bf16 without further loss.

The five workload recipes mirror the paper's settings in shape only: sentence-length
sources for grammatical-error correction and translation, a 400-token source for
summarisation, a joint 32K vocabulary, block size 25 for the drafter-based mode and
batches of at most 32 (Sections 4.1.1, 4.2.1, 4.2.4 and 4.3 of the paper).  The paper's
datasets and trained models are replaced by random weights and by an imposed per-token
agreement rate between draft and greedy output.
"""
from __future__ import annotations

from dataclasses import dataclass, asdict

import numpy as np

MASTER_SEED = 20220510

BOS, PAD, EOS, MASK = 0, 1, 2, 3
FIRST_ORDINARY_ID = 4


@dataclass(frozen=True)
class ModelShape:
    name: str
    d_model: int
    n_heads: int
    d_ffn: int
    vocab: int
    n_enc: int
    n_dec: int
    dtype: str  # "fp32" or "bf16"

    def as_dict(self):
        return asdict(self)


TINY = ModelShape("tiny", 128, 4, 512, 1000, 2, 2, "fp32")
BASE = ModelShape("base", 512, 8, 2048, 32000, 6, 6, "bf16")
BIG = ModelShape("big", 1024, 16, 4096, 32000, 6, 6, "bf16")
# Further shapes the paper reports on (Section 4.1.2: a 12-layer encoder with a 2-layer decoder; Section 4.2.4:
# models of the size of BART-base); same kernels, other layer counts and widths.
DEEP_ENC = ModelShape("deep_encoder_12_2", 512, 8, 2048, 32000, 12, 2, "bf16")
BART_BASE_SIZED = ModelShape("bart_base_sized", 768, 12, 3072, 50265, 6, 6, "bf16")
# A small bf16 shape for fast tests of the tensor-core path (not one of the five workloads).
MINI_BF16 = ModelShape("mini_bf16", 256, 4, 512, 2048, 2, 2, "bf16")


@dataclass(frozen=True)
class Workload:
    index: int          # 1..5, position in the list of configurations
    shape: ModelShape
    mode: str           # "IAD" or "GAD"
    batch: int
    n_batches: int      # how many batches (sentences when batch == 1) make one pass
    src_len_lo: int
    src_len_hi: int     # inclusive
    max_out: int        # 0 = "same as the row's source length"
    k: int              # block size cap
    agreement: float    # per-token draft/greedy agreement; <0 = drafts come from the method itself
    has_drafter: bool


WORKLOADS = {
    1: Workload(1, TINY, "IAD", 1, 1, 16, 16, 24, 17, -1.0, False),
    2: Workload(2, BASE, "IAD", 1, 64, 12, 40, 0, 64, 0.9, False),
    3: Workload(3, BASE, "IAD", 32, 1, 10, 64, 0, 64, 0.9, False),
    4: Workload(4, BIG, "GAD", 1, 32, 20, 50, 0, 25, 0.8, True),
    5: Workload(5, BASE, "GAD", 8, 1, 400, 400, 80, 25, 0.6, True),
}


def _rng(*key: int) -> np.random.Generator:
    return np.random.default_rng(np.random.SeedSequence([MASTER_SEED, *key]))


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bfloat16 (ties to even); result stays float32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    u = (u + 0x7FFF + lsb) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(a.shape)


def _attn_names(prefix):
    return [f"{prefix}.q", f"{prefix}.k", f"{prefix}.v", f"{prefix}.o"]


def weight_names(shape: ModelShape):
    """Ordered (name, array-shape) list of every tensor of one encoder-decoder model."""
    d, F, V = shape.d_model, shape.d_ffn, shape.vocab
    out = [("emb", (V, d))]

    def lin(n, i, o):
        out.append((n + ".W", (i, o)))
        out.append((n + ".b", (o,)))

    def ln(n):
        out.append((n + ".g", (d,)))
        out.append((n + ".b", (d,)))

    for l in range(shape.n_enc):
        for n in _attn_names(f"enc.{l}.self"):
            lin(n, d, d)
        ln(f"enc.{l}.ln1")
        lin(f"enc.{l}.ffn1", d, F)
        lin(f"enc.{l}.ffn2", F, d)
        ln(f"enc.{l}.ln2")
    for l in range(shape.n_dec):
        for n in _attn_names(f"dec.{l}.self"):
            lin(n, d, d)
        ln(f"dec.{l}.ln1")
        for n in _attn_names(f"dec.{l}.cross"):
            lin(n, d, d)
        ln(f"dec.{l}.ln2")
        lin(f"dec.{l}.ffn1", d, F)
        lin(f"dec.{l}.ffn2", F, d)
        ln(f"dec.{l}.ln3")
    return out


def make_weights(shape: ModelShape, model_id: int = 0, std: float = 0.02) -> dict:
    """All tensors ~ N(0, std); LayerNorm gains are 1 + N(0, std).

    ``model_id`` 0 is the autoregressive verifier, 1 the non-autoregressive drafter
    (separate weights of the same shapes).
    """
    shape_key = sum(ord(c) * (i + 1) for i, c in enumerate(shape.name))
    rng = _rng(1000, shape_key, model_id)
    w = {}
    for name, shp in weight_names(shape):
        a = rng.standard_normal(shp, dtype=np.float32) * np.float32(std)
        if name.endswith(".g"):
            a = a + np.float32(1.0)
        if shape.dtype == "bf16":
            a = round_to_bf16(a)
        w[name] = np.ascontiguousarray(a, dtype=np.float32)
    return w


def make_sources(wl: Workload, batch_index: int = 0, vocab: int | None = None):
    """Returns (src [B, Smax] int32 right-padded with PAD, src_len [B] int32)."""
    V = vocab if vocab is not None else wl.shape.vocab
    rng = _rng(2000, wl.index, batch_index)
    lens = rng.integers(wl.src_len_lo, wl.src_len_hi + 1, size=wl.batch).astype(np.int32)
    smax = int(wl.src_len_hi)
    src = np.full((wl.batch, smax), PAD, dtype=np.int32)
    for b in range(wl.batch):
        src[b, : lens[b]] = rng.integers(FIRST_ORDINARY_ID, V, size=int(lens[b]))
    return src, lens


def max_out_lens(wl: Workload, src_len: np.ndarray) -> np.ndarray:
    if wl.max_out > 0:
        return np.full_like(src_len, wl.max_out)
    return src_len.copy()


def corrupt_stream(greedy: np.ndarray, greedy_len: np.ndarray, agreement: float, vocab: int,
                   wl_index: int, batch_index: int = 0) -> np.ndarray:
    """Position-aligned draft stream: each token of a finished greedy output is replaced,
    independently with probability 1 - agreement, by a uniform ordinary id different from it.

    ``greedy`` is [B, T] int32, ``greedy_len`` [B]; positions past a row's length are left as is.
    """
    rng = _rng(3000, wl_index, batch_index)
    g = np.array(greedy, dtype=np.int32, copy=True)
    B, T = g.shape
    flip = rng.random((B, T)) >= agreement
    repl = rng.integers(FIRST_ORDINARY_ID, vocab - 1, size=(B, T)).astype(np.int32)
    repl = np.where(repl >= g, repl + 1, repl)  # uniform over ordinary ids != original
    repl = np.minimum(repl, vocab - 1)
    for b in range(B):
        n = int(greedy_len[b])
        m = flip[b, :n]
        g[b, :n] = np.where(m, repl[b, :n], g[b, :n])
    return g


def random_block_inputs(vocab: int, batch: int, k: int, seed: int):
    """Uniform ordinary token ids [batch, k] for fixed-shape microbenchmarks."""
    rng = _rng(4000, seed)
    return rng.integers(FIRST_ORDINARY_ID, vocab, size=(batch, k)).astype(np.int32)

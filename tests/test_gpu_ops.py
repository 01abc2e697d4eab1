"""Operator-level parity through the C ABI: the two GEMM kernels and the fused projection + arg-max against
the CPU checker's linear map, at sizes that span several tiles and a ragged tail."""
import numpy as np
import pytest
import torch

from oracle import ad_oracle as O
from paper_2205_10350_b200 import binding, synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
OPS = O.Ops("f32")


def _data(M, K, N, bf16, seed=0):
    r = np.random.default_rng(seed)
    x = r.standard_normal((M, K)).astype(np.float32)
    W = (r.standard_normal((N, K)) * 0.1).astype(np.float32)
    b = r.standard_normal(N).astype(np.float32)
    if bf16:
        x, W = synth.round_to_bf16(x), synth.round_to_bf16(W)
    return x, W, b


@pytest.mark.parametrize("M,K,N", [(1, 128, 128), (5, 128, 130), (33, 96, 1000), (17, 512, 257)])
def test_fp32_linear(M, K, N):
    x, W, b = _data(M, K, N, False)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    y = binding.linear(torch.tensor(x, device=DEV), torch.tensor(W, device=DEV), torch.tensor(b, device=DEV), st)
    ref = OPS.linear(x, W.T.copy(), b)
    assert np.abs(y.cpu().numpy() - ref).max() < 1e-4
    assert int(st.item()) == 0


@pytest.mark.parametrize("M,K,N", [(1, 64, 128), (16, 64, 128), (64, 512, 1536), (25, 1024, 300), (200, 512, 512),
                                   (256, 2048, 640), (7, 4096, 128), (100, 2048, 384), (100, 192, 256),
                                   (12, 320, 20000),
                                   # K loops of several ring rounds with more CTAs than SMs (short rings): 4 stages x 4
                                   # rounds and x 6 rounds with four issuers, a depth that would be 5 without the
                                   # divisibility rule, 8 stages x 8 rounds
                                   (64, 1024, 19200), (40, 1536, 19200), (16, 2048, 19200), (64, 4096, 256)])
def test_bf16_tensor_core_linear(M, K, N):
    """Inputs are BF16-exact, the accumulator is FP32: only the summation order differs from the checker.
    The shapes walk through the kernel's configurations: one, two and four MMA issuers, K loops of one and of
    several ring rounds, one and two CTAs per SM, ragged token and feature tiles."""
    x, W, b = _data(M, K, N, True)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    y = binding.linear(torch.tensor(x, device=DEV).bfloat16(), torch.tensor(W, device=DEV).bfloat16(),
                       torch.tensor(b, device=DEV), st)
    ref = OPS.linear(x, W.T.copy(), b)
    assert np.abs(y.cpu().numpy() - ref).max() < 2e-4 * max(1.0, np.abs(ref).max())
    assert int(st.item()) == 0


@pytest.mark.parametrize("bf16,M,d,V", [(False, 9, 128, 1000), (True, 40, 512, 32000), (True, 64, 1024, 4100),
                                        (True, 1, 512, 32000), (True, 130, 256, 2048),
                                        # many tokens (token-stationary kernel): ragged last vocabulary tile, then a
                                        # vocabulary whose last 256-row pair has an empty second half; ragged token tile
                                        (True, 1000, 256, 5000), (True, 1000, 256, 4900), (True, 300, 512, 32000)])
def test_projection_with_fused_argmax(bf16, M, d, V):
    r = np.random.default_rng(4)
    x = r.standard_normal((M, d)).astype(np.float32)
    E = (r.standard_normal((V, d)) * 0.02).astype(np.float32)
    if bf16:
        x, E = synth.round_to_bf16(x), synth.round_to_bf16(E)
    tx, tE = torch.tensor(x, device=DEV), torch.tensor(E, device=DEV)
    if bf16:
        tx, tE = tx.bfloat16(), tE.bfloat16()
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    got = binding.vocab_argmax(tx, tE, st).cpu().numpy()
    lg = OPS.linear(x, E.T.copy(), None)
    for m in range(M):
        i1, v1, i2, v2 = OPS.top2(lg[m])
        if v1 - v2 > 1e-4:
            assert got[m] == i1
        else:
            assert got[m] in (i1, i2)
    assert int(st.item()) == 0


def test_argmax_ties_go_to_the_lowest_id():
    d, V, M = 128, 700, 3
    x = np.ones((M, d), np.float32)
    E = np.zeros((V, d), np.float32)
    E[[650, 131, 400]] = 0.5           # three identical best rows in different 128-row tiles
    got = binding.vocab_argmax(torch.tensor(x, device=DEV), torch.tensor(E, device=DEV)).cpu().numpy()
    assert (got == 131).all()
    got = binding.vocab_argmax(torch.tensor(x, device=DEV).bfloat16(), torch.tensor(E, device=DEV).bfloat16()).cpu().numpy()
    assert (got == 131).all()


def test_tensor_regime_sizes_on_sampled_rows():
    """2048 packed tokens (batch 32 x block 64 of the base model), the size the batched benchmark point runs at:
    256-token tiles, two CTAs per SM, several waves.  The checker computes a sample of token rows (first and last rows
    of tiles, the last row of the pass) of the QKV-sized and FFN-sized projections and of the fused projection +
    arg-max."""
    M, d, V = 2048, 512, 32000
    rows = np.array([0, 1, 127, 128, 255, 256, 1023, 1024, 1500, 1791, 1792, 2046, 2047])
    for (K, N) in ((d, 3 * d), (d, 4 * d), (4 * d, d)):
        x, W, b = _data(M, K, N, True, seed=K + N)
        st = torch.zeros(1, dtype=torch.int32, device=DEV)
        y = binding.linear(torch.tensor(x, device=DEV).bfloat16(), torch.tensor(W, device=DEV).bfloat16(),
                           torch.tensor(b, device=DEV), st).cpu().numpy()
        ref = OPS.linear(x[rows].copy(), W.T.copy(), b)
        assert np.abs(y[rows] - ref).max() < 2e-4 * max(1.0, np.abs(ref).max())
        assert int(st.item()) == 0 and np.isfinite(y).all()
    r = np.random.default_rng(11)
    x = synth.round_to_bf16(r.standard_normal((M, d)).astype(np.float32))
    E = synth.round_to_bf16((r.standard_normal((V, d)) * 0.02).astype(np.float32))
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    got = binding.vocab_argmax(torch.tensor(x, device=DEV).bfloat16(), torch.tensor(E, device=DEV).bfloat16(), st).cpu().numpy()
    assert got.shape == (M,) and int(st.item()) == 0 and (got >= 0).all() and (got < V).all()
    lg = OPS.linear(x[rows].copy(), E.T.copy(), None)
    for j, m in enumerate(rows):
        i1, v1, i2, v2 = OPS.top2(lg[j])
        assert got[m] == i1 if v1 - v2 > 1e-4 else got[m] in (i1, i2)

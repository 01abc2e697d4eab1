"""Pins of the CPU checker's elementary maps against closed forms, brute force and library routines."""
import numpy as np
import pytest
import torch

from oracle import ad_oracle as O

rng = np.random.default_rng(7)


@pytest.fixture(scope="module", params=["f32", "f64"])
def ops(request):
    return O.Ops(request.param)


def tol(ops, f32, f64):
    return f32 if ops.dt == np.float32 else f64


def test_linear_identity_and_one_hot(ops):
    x = rng.standard_normal((5, 7))
    y = ops.linear(x, np.eye(7), np.zeros(7))
    assert np.array_equal(y, x.astype(ops.dt))
    W = rng.standard_normal((7, 3))
    b = rng.standard_normal(3)
    onehot = np.eye(7)[[4, 0]]
    y = ops.linear(onehot, W, b)
    # a one-hot input selects one row of W (so W is [in, out], not its transpose)
    assert np.allclose(y, W[[4, 0]] + b, atol=tol(ops, 1e-6, 1e-14))


def test_linear_matches_library_matmul(ops):
    x = rng.standard_normal((9, 130))
    W = rng.standard_normal((130, 70))
    b = rng.standard_normal(70)
    y = ops.linear(x, W, b)
    assert np.allclose(y, x @ W + b, atol=tol(ops, 2e-4, 1e-11))
    y0 = ops.linear(x, W, None)
    assert np.allclose(y0, x @ W, atol=tol(ops, 2e-4, 1e-11))


def test_layernorm_closed_forms(ops):
    x = rng.standard_normal((4, 64)) * 3 + 5
    y = ops.layernorm(x, np.ones(64), np.zeros(64), eps=0.0)
    assert np.allclose(y.mean(1), 0, atol=tol(ops, 1e-5, 1e-12))
    assert np.allclose(y.var(1), 1, atol=tol(ops, 1e-4, 1e-12))   # biased variance -> exactly 1
    # constant row: zero variance, only eps keeps it finite, output = beta
    c = np.full((1, 64), 2.5)
    beta = rng.standard_normal(64)
    assert np.allclose(ops.layernorm(c, np.ones(64), beta, eps=1e-5), beta, atol=1e-6)


def test_layernorm_matches_library(ops):
    x = rng.standard_normal((6, 48))
    g = rng.standard_normal(48)
    b = rng.standard_normal(48)
    ref = torch.nn.functional.layer_norm(torch.tensor(x), (48,), torch.tensor(g), torch.tensor(b), 1e-5).numpy()
    assert np.allclose(ops.layernorm(x, g, b, 1e-5), ref, atol=tol(ops, 1e-5, 1e-12))


def brute_attention(q, k, v, limit, H):
    Mq, d = q.shape
    dh = d // H
    out = np.zeros((Mq, d))
    for i in range(Mq):
        for h in range(H):
            mask = np.full(k.shape[0], -np.inf)
            mask[: limit[i]] = 0.0
            s = np.array([sum(q[i, h * dh + c] * k[j, h * dh + c] for c in range(dh)) for j in range(k.shape[0])])
            s = s / np.sqrt(dh) + mask
            p = np.exp(s - s.max())
            p = p / p.sum()
            assert abs(p.sum() - 1) < 1e-12
            for c in range(dh):
                out[i, h * dh + c] = sum(p[j] * v[j, h * dh + c] for j in range(k.shape[0]))
    return out


@pytest.mark.parametrize("case", ["block_causal_offset", "non_causal", "key_padding"])
def test_attention_brute_force(ops, case):
    H, d, Mq, Mk = 2, 8, 4, 7
    q = rng.standard_normal((Mq, d))
    k = rng.standard_normal((Mk, d))
    v = rng.standard_normal((Mk, d))
    if case == "block_causal_offset":      # prefix of 3 cached positions, query i sees 0..3+i
        lim = [3 + i + 1 for i in range(Mq)]
    elif case == "non_causal":
        lim = [Mk] * Mq
    else:                                    # only the first 5 keys are real
        lim = [5] * Mq
    got = ops.attention(q, k, v, lim, H)
    assert np.allclose(got, brute_attention(q, k, v, lim, H), atol=tol(ops, 1e-5, 1e-12))


def test_attention_matches_library_sdpa(ops):
    H, d, M = 4, 32, 6
    q, k, v = (rng.standard_normal((M, d)) for _ in range(3))
    lim = [i + 1 for i in range(M)]
    tq, tk, tv = (torch.tensor(a).view(M, H, d // H).transpose(0, 1) for a in (q, k, v))
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)
    ref = ref.transpose(0, 1).reshape(M, d).numpy()
    assert np.allclose(ops.attention(q, k, v, lim, H), ref, atol=tol(ops, 1e-5, 1e-12))


def test_attention_uniform_when_queries_are_zero(ops):
    H, d, Mk = 2, 8, 5
    v = rng.standard_normal((Mk, d))
    k = rng.standard_normal((Mk, d))
    out = ops.attention(np.zeros((1, d)), k, v, [4], H)
    assert np.allclose(out[0], v[:4].mean(0), atol=tol(ops, 1e-6, 1e-13))


def test_top2_and_ties(ops):
    i1, v1, i2, v2 = ops.top2(np.array([0.5, 2.0, -1.0, 2.0, 1.5]))
    assert (i1, v1) == (1, 2.0)            # lowest id wins the tie
    assert (i2, v2) == (3, 2.0)
    i1, v1, i2, v2 = ops.top2(np.array([3.0, 1.0, 2.0]))
    assert (i1, i2) == (0, 2)
    i1, v1, i2, v2 = ops.top2(np.array([1.0, 2.0, 3.0]))
    assert (i1, i2) == (2, 1)

"""Pins of the decode-attention oracle (paper Section V-B): closed forms, a library softmax, brute force,
and the exactness of the partitioned execution with anchors for any partition count and merge order."""
import itertools
import math

import numpy as np
import pytest
from scipy.special import softmax

from oracle.attention import decode_attention, decode_attention_partitioned, merge_partials, partial_attention


def _case(seed, B=3, Hq=4, Hkv=2, L=37, d=16):
    rng = np.random.default_rng(seed)
    q = rng.standard_normal((B, Hq, d))
    K = rng.standard_normal((B, Hkv, L, d))
    V = rng.standard_normal((B, Hkv, L, d))
    kv_len = rng.integers(1, L + 1, size=B)
    return q, K, V, kv_len


def test_closed_forms():
    q, K, V, _ = _case(1)
    L = K.shape[2]
    full = np.full(3, L)
    # a single token: the output is its value row
    one = decode_attention(q, K, V, np.ones(3, int), 0.25)
    assert np.allclose(one, np.repeat(V[:, :, 0], 2, axis=1), atol=1e-15)
    # a zero query scores every token alike: the mean of the value rows
    mean = decode_attention(np.zeros_like(q), K, V, full, 0.25)
    assert np.allclose(mean, np.repeat(V.mean(axis=2), 2, axis=1), atol=1e-14)
    # weights sum to one: constant values come back unchanged
    assert np.allclose(decode_attention(q, K, np.ones_like(V), full, 0.25), 1.0, atol=1e-14)
    # one overwhelming score picks that token's value row
    K2 = K.copy()
    K2[:, :, 5] = 0
    K2[0, 0, 5] = 200 * q[0, 0] / np.dot(q[0, 0], q[0, 0])
    got = decode_attention(q, K2, V, full, 1.0)
    assert np.allclose(got[0, 0], V[0, 0, 5], atol=1e-12)
    # an empty cache leaves a zero row, tokens beyond kv_len are never read
    lens = np.array([0, 4, L])
    K3, V3 = K.copy(), V.copy()
    K3[1, :, 4:], V3[1, :, 4:] = np.nan, np.nan
    out = decode_attention(q, K3, V3, lens, 0.25)
    assert np.all(out[0] == 0) and np.all(np.isfinite(out))


def test_matches_a_library_softmax_and_brute_force():
    q, K, V, kv_len = _case(2)
    scale = 1 / math.sqrt(q.shape[2])
    got = decode_attention(q, K, V, kv_len, scale)
    for b, h in itertools.product(range(3), range(4)):
        L = kv_len[b]
        w = softmax(scale * K[b, h // 2, :L] @ q[b, h])
        assert np.allclose(got[b, h], w @ V[b, h // 2, :L], atol=1e-14)
    # brute force, scalar loops, one (request, head)
    b, h = 1, 3
    L = int(kv_len[b])
    scores = [scale * sum(q[b, h, i] * K[b, 1, t, i] for i in range(16)) for t in range(L)]
    z = sum(math.exp(s) for s in scores)
    want = [sum(math.exp(scores[t]) / z * V[b, 1, t, j] for t in range(L)) for j in range(16)]
    assert np.allclose(got[b, h], want, atol=1e-13)


@pytest.mark.parametrize("n_part", [1, 2, 3, 4, 7, 64])
def test_partitioned_execution_is_exact(n_part):
    q, K, V, kv_len = _case(3 + n_part)
    kv_len[0] = 2                      # fewer tokens than partitions: some shares are empty
    scale = 0.3
    want = decode_attention(q, K, V, kv_len, scale)
    got = decode_attention_partitioned(q, K, V, kv_len, scale, n_part)
    assert np.max(np.abs(got - want)) <= 1e-13
    # partial results may come back in any order
    rng = np.random.default_rng(n_part)
    for _ in range(3):
        order = rng.permutation(n_part)
        assert np.max(np.abs(decode_attention_partitioned(q, K, V, kv_len, scale, n_part, order) - want)) <= 1e-13


def test_anchor_is_the_share_maximum_and_merge_rescales():
    rng = np.random.default_rng(9)
    qv, Kh, Vh = rng.standard_normal(8), rng.standard_normal((10, 8)), rng.standard_normal((10, 8))
    a, l, o = partial_attention(qv, Kh, Vh, np.array([1, 4, 7]), 0.5)
    P = 0.5 * Kh[[1, 4, 7]] @ qv
    assert a == P.max() and l == pytest.approx(np.exp(P - P.max()).sum()) and 1.0 <= l <= 3.0
    # two shares whose anchors differ by 1000: naive exponentials overflow, the rescaled merge does not
    big = (1000.0, 1.0, np.array([2.0]))
    small = (0.0, 5.0, np.array([50.0]))
    assert merge_partials([big, small])[0] == pytest.approx(2.0)
    assert merge_partials([small, big])[0] == pytest.approx(2.0)
    assert merge_partials([small, (-np.inf, 0.0, np.zeros(1))])[0] == pytest.approx(10.0)

"""Pins for the attention oracle (oracle/attention.py): closed forms of the rotary embedding,
its group properties, special cases of softmax attention with known answers, and a library
routine for the softmax-weighted sum.  Never the CUDA path."""
import math

import numpy as np
import pytest
import torch

from oracle import attention as oa

TOL = 1e-11


def rng(seed):
    return np.random.default_rng(seed)


def test_rope_two_channels_is_a_plane_rotation():
    # d = 2: one pair, angle = pos * base^0 = pos; a quarter turn maps (1, 0) to (0, 1)
    assert np.allclose(oa.rope([1.0, 0.0], math.pi / 2, 10000.0), [0.0, 1.0], atol=1e-15)
    assert np.allclose(oa.rope([0.0, 1.0], math.pi / 2, 10000.0), [-1.0, 0.0], atol=1e-15)
    assert np.allclose(oa.rope([2.0, 3.0], math.pi, 7.0), [-2.0, -3.0], atol=1e-14)


def test_rope_pairs_channel_c_with_c_plus_half_and_slows_down_with_c():
    # d = 4, base = 100: pair 0 = channels (0, 2) turns by pos, pair 1 = channels (1, 3) by pos / 10
    x = np.array([1.0, 1.0, 0.0, 0.0])
    y = oa.rope(x, 0.3, 100.0)
    assert np.allclose(y, [math.cos(0.3), math.cos(0.03), math.sin(0.3), math.sin(0.03)], atol=1e-15)


def test_rope_identity_composition_norm_and_switch():
    x = rng(1).standard_normal((5, 128))
    assert np.array_equal(oa.rope(x, 0, 10000.0), x)
    assert np.array_equal(oa.rope(x, 17, 0.0), x)
    assert np.allclose(oa.rope(oa.rope(x, 5, 10000.0), 12, 10000.0), oa.rope(x, 17, 10000.0), atol=1e-12)
    assert np.allclose(np.linalg.norm(oa.rope(x, 99, 500000.0), axis=-1), np.linalg.norm(x, axis=-1), rtol=1e-13)


def test_rope_scores_depend_on_relative_position_only():
    r = rng(2)
    q, k = r.standard_normal(64), r.standard_normal(64)
    a = np.dot(oa.rope(q, 40, 10000.0), oa.rope(k, 33, 10000.0))
    b = np.dot(oa.rope(q, 1007, 10000.0), oa.rope(k, 1000, 10000.0))
    c = np.dot(oa.rope(q, 7, 10000.0), k)
    assert abs(a - b) < 1e-10 and abs(a - c) < 1e-10


def test_equal_keys_give_the_mean_of_the_values():
    r = rng(3)
    V = r.standard_normal((10, 8))
    K = np.tile(r.standard_normal((1, 8)), (10, 1))
    out = oa.attend_decode(r.standard_normal((2, 8)), K, V, 7, 0.0)   # RoPE off: all 7 scores equal
    assert np.allclose(out, np.tile(V[:7].mean(axis=0), (2, 1)), atol=1e-13)


def test_one_dominant_key_returns_its_value_and_length_bounds_the_rows():
    d = 16
    K = np.zeros((6, d))
    V = rng(4).standard_normal((6, d))
    q = np.zeros((1, d))
    q[0, 0] = 1.0
    K[2, 0] = 400.0   # score 100 against 0 elsewhere
    K[5, 0] = 4000.0  # beyond `length`: must be ignored
    out = oa.attend_decode(q, K, V, 5, 0.0)
    assert np.allclose(out[0], V[2], atol=1e-12)
    assert np.allclose(oa.attend_decode(q, K, V, 1, 0.0)[0], V[0], atol=1e-15)  # a single row: weight 1


def test_two_rows_closed_form_with_positions():
    # d = 2, base irrelevant (one pair, angle = position).  Keys (1,0) at rows 0 and 1, query (1,0)
    # at position 1: scores scale * cos(1), scale * cos(0)  ->  softmax of two numbers.
    K = np.array([[1.0, 0.0], [1.0, 0.0]])
    V = np.array([[1.0, 0.0], [0.0, 1.0]])
    out = oa.attend_decode(np.array([[1.0, 0.0]]), K, V, 2, 10000.0, scale=2.0)
    w0 = 1.0 / (1.0 + math.exp(2.0 * (1.0 - math.cos(1.0))))
    assert np.allclose(out[0], [w0, 1.0 - w0], atol=1e-14)


@pytest.mark.parametrize("G,length,d,base", [(1, 1, 8, 10000.0), (4, 37, 128, 10000.0), (2, 300, 64, 500000.0)])
def test_softmax_weighted_sum_matches_library(G, length, d, base):
    """The library computes softmax(q k^T * scale) v; the rotary embedding is applied beforehand
    with a complex multiplication, a different route to the same rotation."""
    r = rng(length)
    q, K, V = r.standard_normal((G, d)), r.standard_normal((length + 3, d)), r.standard_normal((length + 3, d))

    def rot(x, pos):
        h = d // 2
        z = (x[..., :h] + 1j * x[..., h:]) * np.exp(1j * pos * base ** (-2.0 * np.arange(h) / d))
        return np.concatenate([z.real, z.imag], axis=-1)

    qr = np.stack([rot(q[g], length - 1) for g in range(G)])
    kr = np.stack([rot(K[j], j) for j in range(length)])
    want = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(qr)[None], torch.from_numpy(kr)[None], torch.from_numpy(V[:length])[None]).numpy()[0]
    got = oa.attend_decode(q, K, V, length, base)
    assert np.linalg.norm(got - want) / np.linalg.norm(want) < TOL


def test_output_is_a_convex_combination_of_the_value_rows():
    r = rng(9)
    V = r.standard_normal((50, 12))
    out = oa.attend_decode(r.standard_normal((3, 12)) * 3, r.standard_normal((50, 12)), V, 50, 10000.0)
    assert np.all(out <= V.max(axis=0) + 1e-12) and np.all(out >= V.min(axis=0) - 1e-12)


# ---- chunk-wise prefilling (Section 3.3): every token of a chunk, causally ----

def test_prefill_of_one_token_is_the_decoding_step():
    r = rng(31)
    K, V, q = r.standard_normal((40, 16)), r.standard_normal((40, 16)), r.standard_normal((2, 1, 16))
    assert np.array_equal(oa.attend_prefill(q, K, V, 33, 10000.0), oa.attend_decode(q[:, 0], K, V, 33, 10000.0)[:, None, :])


def test_prefill_is_causal_and_ignores_rows_past_the_length():
    r = rng(32)
    K, V, q = r.standard_normal((30, 8)), r.standard_normal((30, 8)), r.standard_normal((1, 5, 8))
    base = oa.attend_prefill(q, K, V, 20, 10000.0)
    K2, V2 = K.copy(), V.copy()
    K2[18:], V2[18:] = 7.0, -3.0           # rows of chunk tokens 3, 4 and everything after the cache length
    got = oa.attend_prefill(q, K2, V2, 20, 10000.0)
    assert np.array_equal(got[:, :3], base[:, :3])   # tokens 0..2 see rows 0..17 only
    assert not np.allclose(got[:, 3:], base[:, 3:])


def test_prefill_first_token_of_an_empty_history_returns_its_own_value():
    r = rng(33)
    K, V, q = r.standard_normal((6, 4)), r.standard_normal((6, 4)), r.standard_normal((3, 6, 4))
    out = oa.attend_prefill(q, K, V, 6, 10000.0)      # the chunk is the whole cache: token 0 sees row 0 only
    assert np.allclose(out[:, 0], np.broadcast_to(V[0], (3, 4)), atol=TOL)


def test_prefill_matches_masked_matrix_softmax_without_rope():
    # no RoPE: the textbook causal attention softmax(mask(Q K^T / sqrt d)) V with the chunk at the end
    r = rng(34)
    n, length, d = 7, 19, 8
    K, V, q = r.standard_normal((25, d)), r.standard_normal((25, d)), r.standard_normal((2, n, d))
    scores = torch.from_numpy(q) @ torch.from_numpy(K[:length]).T / math.sqrt(d)
    rows = torch.arange(length)[None, :] <= (length - n + torch.arange(n))[:, None]
    want = torch.softmax(scores.masked_fill(~rows, float("-inf")), dim=-1) @ torch.from_numpy(V[:length])
    assert np.allclose(oa.attend_prefill(q, K, V, length, 0.0), want.numpy(), atol=TOL)


def test_prefill_with_rope_matches_matrix_form():
    # RoPE at in-cache positions written as matrices: rotate every key row by its index, every query by its row index
    r = rng(35)
    n, length, d, base = 4, 11, 16, 10000.0
    K, V, q = r.standard_normal((12, d)), r.standard_normal((12, d)), r.standard_normal((1, n, d))
    Kr = np.stack([oa.rope(K[j], j, base) for j in range(length)])
    Qr = np.stack([oa.rope(q[0, i], length - n + i, base) for i in range(n)])
    S = Qr @ Kr.T / math.sqrt(d)
    for i in range(n):
        S[i, length - n + i + 1:] = -np.inf
    W = np.exp(S - S.max(axis=1, keepdims=True))
    W /= W.sum(axis=1, keepdims=True)
    assert np.allclose(oa.attend_prefill(q, K, V, length, base)[0], W @ V[:length], atol=TOL)

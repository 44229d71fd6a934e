"""Attention over the compressed cache (decoding and chunk-wise prefilling) -- TEST INFRASTRUCTURE,
not part of the product.

Plain fp64 numpy statement of Section 3.4 (the attention of a newly incoming token over sink
tokens, compressed tokens and recent tokens, the second attention equation of that section)
with the position encoding the section prescribes: key states are cached BEFORE RoPE, and when
attention is computed every cached key gets the position index of its row within the cache,
not within the original sequence.  Written with explicit loops over query heads and cache rows
so that it can be checked against the paper by eye.

RoPE itself is the rotary embedding the paper cites: channel pair c of a vector at position p
is rotated by the angle p * base^(-2c/d).  Which two channels form pair c is not fixed by the
paper; the LLaMA models it uses pair channel c with channel c + d/2, and that is what is done
here (a reading, listed as such in the design notes).

Only ``tests/`` and ``__graft_entry__.smoke()`` may import this module.  It imports nothing
from the CUDA package.  Pins: ``tests/test_oracle_attention_pins.py``.
"""
from __future__ import annotations

import numpy as np


def rope(x, pos: float, base: float) -> np.ndarray:
    """Rotary position embedding of one vector (or a stack of vectors, last axis = channels) at
    position ``pos``: (x_c, x_{c+d/2}) -> (x_c cos a - x_{c+d/2} sin a, x_{c+d/2} cos a + x_c sin a),
    a = pos * base^(-2c/d), c = 0 .. d/2 - 1.  ``base <= 0`` switches the embedding off."""
    x = np.asarray(x, dtype=np.float64)
    if base <= 0:
        return x.copy()
    d = x.shape[-1]
    if d % 2:
        raise ValueError("RoPE needs an even number of channels")
    h = d // 2
    c = np.arange(h, dtype=np.float64)
    angle = pos * base ** (-2.0 * c / d)
    cos, sin = np.cos(angle), np.sin(angle)
    out = np.empty_like(x)
    out[..., :h] = x[..., :h] * cos - x[..., h:] * sin
    out[..., h:] = x[..., h:] * cos + x[..., :h] * sin
    return out


def attend_decode(q, k_cache, v_cache, length: int, rope_base: float, scale: float | None = None) -> np.ndarray:
    """Output of the attention of one new token (Section 3.4).

    ``q``: ``[G, d]`` queries (before RoPE) of the G query heads that share this KV head;
    ``k_cache`` / ``v_cache``: ``[capacity, d]`` with rows ``[0, length)`` valid -- sinks,
    compressed rows and recent rows alike, the new token's own key and value in row
    ``length - 1``.  Row j of the key cache gets position j, the query position ``length - 1``;
    scores are scaled by ``scale`` (default 1/sqrt(d)), softmax over the ``length`` rows.
    Returns ``[G, d]`` in fp64.
    """
    q = np.asarray(q, dtype=np.float64)
    K = np.asarray(k_cache, dtype=np.float64)
    V = np.asarray(v_cache, dtype=np.float64)
    G, d = q.shape
    if not 1 <= length <= K.shape[0]:
        raise ValueError("need 1 <= length <= capacity")
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    out = np.zeros((G, d))
    for g in range(G):
        qr = rope(q[g], length - 1, rope_base)
        scores = np.empty(length)
        for j in range(length):
            scores[j] = scale * np.dot(qr, rope(K[j], j, rope_base))
        w = np.exp(scores - scores.max())
        w /= w.sum()
        for j in range(length):
            out[g] += w[j] * V[j]
    return out


def attend_prefill(q, k_cache, v_cache, length: int, rope_base: float, scale: float | None = None) -> np.ndarray:
    """Outputs of the attention of a chunk of incoming tokens (Section 3.3, chunk-wise processing
    during training and prefilling, first attention equation).

    The chunk's ``n`` tokens have been appended to the cache: they sit in rows
    ``[length - n, length)``.  Token i of the chunk attends to the sink rows, the compressed rows,
    the chunk's earlier tokens and itself, i.e. to cache rows ``[0, length - n + i]``; positions
    are the row indices in the cache for keys and query alike.  That is the decoding step of the
    cache as it stood when token i had just been appended, so that is how it is computed.
    ``q``: ``[G, n, d]`` (before RoPE); returns ``[G, n, d]`` in fp64.
    """
    q = np.asarray(q, dtype=np.float64)
    G, n, d = q.shape
    if not 1 <= n <= length:
        raise ValueError("need 1 <= chunk length <= cache length")
    out = np.empty((G, n, d))
    for i in range(n):
        out[:, i, :] = attend_decode(q[:, i, :], k_cache, v_cache, length - n + i + 1, rope_base, scale)
    return out

"""Decode attention as the paper states it (Section V-B), float64, plain numpy.

Test infrastructure, like everything under oracle/: only tests (and the benchmark's CPU leg) may
import it; it shares nothing with the CUDA path.

Two functions:
  decode_attention            the definition: P = q K^T (scaled), S = softmax(P), O = S V, per request
                              and head, over the first kv_len tokens of the request's cache;
  decode_attention_partitioned  the paper's integral execution: the KV cache of a request is dealt out
                              token by token to n_part partitions (token i to partition i mod n_part),
                              every partition runs all three steps on its share with a partial softmax
                              that keeps an anchor (its running maximum), and the partial outputs are
                              rescaled by their anchors into the exact global output, in any order.
Shapes: q [B, Hq, d]; K, V [B, Hkv, Lmax, d]; kv_len [B]; query head h reads KV head h // (Hq // Hkv).
"""
from __future__ import annotations

import numpy as np


def decode_attention(q, K, V, kv_len, scale: float) -> np.ndarray:
    q, K, V = (np.asarray(a, np.float64) for a in (q, K, V))
    B, Hq, d = q.shape
    Hkv = K.shape[1]
    G = Hq // Hkv
    out = np.zeros((B, Hq, d), np.float64)
    for b in range(B):
        L = int(kv_len[b])
        if L == 0:
            continue                                   # nothing to attend to: the output row stays zero
        for h in range(Hq):
            Kh, Vh = K[b, h // G, :L], V[b, h // G, :L]
            P = scale * (Kh @ q[b, h])                 # step 1
            S = np.exp(P - P.max())
            S /= S.sum()                               # step 2 (softmax, shifted by its maximum for range only)
            out[b, h] = S @ Vh                         # step 3
    return out


def partial_attention(q_bh, Kh, Vh, token_ids, scale: float):
    """One partition's share of one (request, head): anchor a = max P_i, l = sum exp(P_i - a),
    o = sum exp(P_i - a) V_i over its tokens; an empty share returns (-inf, 0, 0)."""
    d = q_bh.shape[0]
    if len(token_ids) == 0:
        return -np.inf, 0.0, np.zeros(d, np.float64)
    P = scale * (Kh[token_ids] @ q_bh)
    a = P.max()
    w = np.exp(P - a)
    return a, w.sum(), w @ Vh[token_ids]


def merge_partials(parts):
    """Rescale (anchor, l, o) triples into the global output: O = sum e^(a_p - a) o_p / sum e^(a_p - a) l_p
    with a = max a_p.  The order of `parts` does not matter."""
    a = max(p[0] for p in parts)
    num = sum(np.exp(p[0] - a) * p[2] for p in parts if p[1] > 0)
    den = sum(np.exp(p[0] - a) * p[1] for p in parts if p[1] > 0)
    return num / den


def decode_attention_partitioned(q, K, V, kv_len, scale: float, n_part: int, order=None) -> np.ndarray:
    q, K, V = (np.asarray(a, np.float64) for a in (q, K, V))
    B, Hq, d = q.shape
    G = Hq // K.shape[1]
    out = np.zeros((B, Hq, d), np.float64)
    for b in range(B):
        L = int(kv_len[b])
        if L == 0:
            continue
        shares = [np.arange(p, L, n_part) for p in range(n_part)]      # token i lives in partition i mod n_part
        for h in range(Hq):
            parts = [partial_attention(q[b, h], K[b, h // G], V[b, h // G], ids, scale) for ids in shares]
            if order is not None:
                parts = [parts[i] for i in order]
            out[b, h] = merge_partials(parts)
    return out

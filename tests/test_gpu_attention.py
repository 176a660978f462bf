"""Decode attention on the GPU against the float64 oracle (paper Section V-B), through the C ABI."""
import math

import numpy as np
import pytest
import torch

import paper_2608_05483_b200 as P
from gpu_util import DEV, bits_to_dev
from oracle.attention import decode_attention
from workloads import bf16_bits_to_f64, f32_to_bf16_bits

pytestmark = pytest.mark.gpu

TOL = 2e-5      # fp32 accumulation over a few thousand bf16 products and exponentials; an indexing mistake is far above


def _problem(seed, B, Hkv, G, Lmax, lens=None, poison=True):
    rng = np.random.default_rng(seed)
    d = 128
    q = f32_to_bf16_bits(rng.standard_normal((B, Hkv * G, d), dtype=np.float32))
    K = f32_to_bf16_bits(rng.standard_normal((B, Hkv, Lmax, d), dtype=np.float32))
    V = f32_to_bf16_bits(rng.standard_normal((B, Hkv, Lmax, d), dtype=np.float32))
    kv_len = np.asarray(lens if lens is not None else rng.integers(1, Lmax + 1, size=B), np.int32)
    if poison:   # what lies beyond a request's length must never reach the result: fill it with NaN patterns
        for b in range(B):
            K[b, :, kv_len[b]:] = 0x7FC0
            V[b, :, kv_len[b]:] = 0x7FC0
    return q, K, V, kv_len


def _run(q, K, V, kv_len, scale):
    out, ws = P.attn_decode(bits_to_dev(q), bits_to_dev(K), bits_to_dev(V), torch.from_numpy(kv_len).to(DEV), scale)
    torch.cuda.synchronize()
    rc, status = P.plora_attn_status(ws.data_ptr())
    assert rc == 0 and status == 0
    return out.cpu().numpy()


def _check(q, K, V, kv_len, scale):
    got = _run(q, K, V, kv_len, scale)
    Kc, Vc = K.copy(), V.copy()
    for b in range(len(kv_len)):           # the oracle never reads beyond kv_len either, but numpy would carry the NaNs
        Kc[b, :, kv_len[b]:] = 0
        Vc[b, :, kv_len[b]:] = 0
    ref = decode_attention(bf16_bits_to_f64(q), bf16_bits_to_f64(Kc), bf16_bits_to_f64(Vc), kv_len, scale)
    assert np.all(np.isfinite(got))
    assert np.max(np.abs(got - ref)) <= TOL * max(1.0, np.max(np.abs(ref)))
    return got


@pytest.mark.parametrize("G", [1, 2, 4, 8])
def test_matches_the_oracle(G):
    q, K, V, kv_len = _problem(10 + G, B=5, Hkv=3, G=G, Lmax=700)
    _check(q, K, V, kv_len, 1 / math.sqrt(128))


def test_lengths_around_tile_and_chunk_boundaries():
    lens = [1, 7, 8, 9, 63, 64, 65, 255, 256, 257, 511, 512, 513, 1000, 0, 1024]
    q, K, V, kv_len = _problem(30, B=len(lens), Hkv=2, G=1, Lmax=1024, lens=lens)
    got = _check(q, K, V, kv_len, 0.1)
    assert np.all(got[14] == 0)            # an empty cache leaves a zero row
    # a single token returns its value row (exactly: weight 1)
    assert np.array_equal(got[0], bf16_bits_to_f64(V[0, :, 0]).astype(np.float32))


def test_large_scores_do_not_overflow_and_repeat_bit_for_bit():
    q, K, V, kv_len = _problem(40, B=4, Hkv=4, G=2, Lmax=900)
    first = _check(q, K, V, kv_len, 3.0)   # scores of several hundred: only the anchors keep the exponentials in range
    for _ in range(5):
        assert _run(q, K, V, kv_len, 3.0).tobytes() == first.tobytes()


def test_argument_errors():
    q, K, V, kv_len = _problem(50, B=2, Hkv=2, G=1, Lmax=64)
    qd, Kd, Vd, ld = bits_to_dev(q), bits_to_dev(K), bits_to_dev(V), torch.from_numpy(kv_len).to(DEV)
    out = torch.empty((2, 2, 128), dtype=torch.float32, device=DEV)
    need = P.plora_attn_workspace_bytes(2, 64, 2, 1)
    ws = torch.zeros(need, dtype=torch.uint8, device=DEV)
    args = lambda **kw: P.plora_attn_decode(qd.data_ptr(), Kd.data_ptr(), Vd.data_ptr(), ld.data_ptr(), 2, 64, 2,
                                            kw.get("G", 1), kw.get("d", 128), 0.1, out.data_ptr(), ws.data_ptr(),
                                            kw.get("ws_bytes", need))
    assert args() == 0
    assert args(d=64) == P.ERR_UNSUPPORTED and args(G=3) == P.ERR_UNSUPPORTED
    assert args(ws_bytes=need - 1) == P.ERR_WORKSPACE
    assert P.plora_attn_workspace_bytes(0, 64, 2, 1) == 0
    torch.cuda.synchronize()

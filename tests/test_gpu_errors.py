"""Host-visible error paths: every one returns a status before anything is launched."""
import numpy as np
import pytest
import torch

import paper_2608_05483_b200 as P
from gpu_util import DEV, Runner
from helpers import random_problem


def load_raw():
    return P.load()

pytestmark = pytest.mark.gpu


def test_error_statuses():
    p = random_problem(3, T=8, d_in=64, d_out=64, ranks=[8, 8])
    r = Runner(p, max_tokens=8)
    h = r.ctx.handle
    y = torch.zeros((8, 64), dtype=torch.float32, device=DEV)
    n0 = r.ctx.launch_count()
    x, ids = r.x.data_ptr(), r.ids.data_ptr()
    assert P.plora_lora_delta(h, 0, ids, 8, 0, 0, y.data_ptr()) == P.ERR_INVALID_ARG
    assert P.plora_lora_delta(h, x, 0, 8, 0, 0, y.data_ptr()) == P.ERR_INVALID_ARG
    assert P.plora_lora_delta(h, x, ids, 8, 0, 0, 0) == P.ERR_INVALID_ARG
    assert P.plora_lora_delta(h, x, ids, -1, 0, 0, y.data_ptr()) == P.ERR_INVALID_ARG
    assert P.plora_lora_delta(h, x, ids, 9, 0, 0, y.data_ptr()) == P.ERR_INVALID_ARG       # above max_tokens
    assert P.plora_lora_delta(h, x + 2, ids, 8, 0, 0, y.data_ptr()) == P.ERR_INVALID_ARG   # misaligned x
    assert P.plora_lora_delta(h, x, ids, 8, 5, 0, y.data_ptr()) == P.ERR_NOT_REGISTERED
    assert P.plora_bucket(h, ids, 8, 0) == P.ERR_INVALID_ARG
    assert P.plora_bucket(h, ids, 8, 3) == P.ERR_INVALID_ARG                               # above max_adapters
    assert P.plora_pool_max_rank(h, 9, 9) == P.ERR_NOT_REGISTERED
    m = torch.zeros((8, 4), dtype=torch.float32, device=DEV)
    assert P.plora_shrink(h, x, ids, 8, 0, 0, m.data_ptr(), 4) == P.ERR_INVALID_ARG        # ldm below the padded rank
    assert P.plora_set_path(h, 17, 0) == P.ERR_INVALID_ARG
    assert load_raw().plora_set_inputs_resident(None, 1) == P.ERR_INVALID_ARG
    assert load_raw().plora_set_inputs_resident(h, 2) == P.ERR_INVALID_ARG
    assert P.plora_set_inputs_resident(h, True) == P.OK and P.plora_set_inputs_resident(h, False) == P.OK
    assert r.ctx.launch_count() == n0
    assert P.plora_lora_delta(h, x, ids, 0, 0, 0, y.data_ptr()) == P.OK                   # empty batch is fine
    r.close()


def test_register_errors():
    ctx = P.Context(8, 2)
    ranks = np.array([8, 8], np.int32)
    scales = np.ones(2, np.float32)
    A = [np.zeros((64, 8), np.uint16)] * 2
    B = [np.zeros((8, 64), np.uint16)] * 2
    slab = ctx.register_pool(0, 0, 64, 64, ranks, scales, A, B)
    import ctypes
    pa = (ctypes.c_void_p * 2)(A[0].ctypes.data, A[1].ctypes.data)
    pb = (ctypes.c_void_p * 2)(B[0].ctypes.data, B[1].ctypes.data)
    d = P.PoolDesc(0, 1, 64, 64, 2, 0, ranks.ctypes.data, scales.ctypes.data, ctypes.cast(pa, ctypes.c_void_p).value,
                   ctypes.cast(pb, ctypes.c_void_p).value)
    assert P.plora_register_pool(ctx.handle, d, slab.data_ptr(), 16, 0) == P.ERR_WORKSPACE      # slab too small
    assert P.plora_register_pool(ctx.handle, d, 0, slab.numel(), 0) == P.ERR_INVALID_ARG
    d3 = P.PoolDesc(0, 1, 64, 64, 3, 0, ranks.ctypes.data, scales.ctypes.data, None, None)
    assert P.plora_register_pool(ctx.handle, d3, slab.data_ptr(), slab.numel(), 0) == P.ERR_INVALID_ARG
    with pytest.raises(P.PloraError):
        ctx.register_pool(0, 2, 60, 64, ranks, scales, [np.zeros((60, 8), np.uint16)] * 2, B)    # d_in not a multiple of 8
    ctx.close()


def test_reregistration_replaces_the_pool():
    p = random_problem(8, T=6, d_in=64, d_out=64, ranks=[8, 8])
    r = Runner(p)
    first = r.delta(P.PATH_FUSED)
    zB = [np.zeros_like(b) for b in p["B"]]
    r.slab = r.ctx.register_pool(0, 0, 64, 64, p["ranks"], p["scales"], p["A"], zB)
    assert np.all(r.delta(P.PATH_FUSED) == 0) and np.any(first != 0)
    r.close()


def test_read_bandwidth_probe():
    # the probe folds what it reads into per-block checksums: their XOR is the XOR of all words of the buffer
    n = (8 << 20) + 4096 + 16                      # not a multiple of the kernel's stride: the tail loop runs too
    buf = torch.randint(-2**31, 2**31 - 1, (n // 4,), dtype=torch.int32, device=DEV)
    sink = torch.zeros(1 << 14, dtype=torch.int32, device=DEV)
    assert P.plora_stream_read(buf.data_ptr(), n, sink.data_ptr(), sink.numel() * 4) == P.OK
    torch.cuda.synchronize()
    want = np.bitwise_xor.reduce(buf.cpu().numpy().view(np.uint32))
    got = np.bitwise_xor.reduce(sink.cpu().numpy().view(np.uint32))
    assert got == want
    assert P.plora_stream_read(buf.data_ptr(), n, sink.data_ptr(), 16) == P.ERR_WORKSPACE        # sink too small
    assert P.plora_stream_read(buf.data_ptr() + 4, n - 16, sink.data_ptr(), 1 << 16) == P.ERR_INVALID_ARG
    assert P.plora_stream_read(buf.data_ptr(), n - 8, sink.data_ptr(), 1 << 16) == P.ERR_INVALID_ARG
    assert P.plora_stream_read(0, n, sink.data_ptr(), 1 << 16) == P.ERR_INVALID_ARG

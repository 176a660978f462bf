"""The allocation-free entry point, plora_lora_delta_noalloc, against plora_lora_delta.

It serves hosts that cannot call cudaMalloc where they need the delta (a serving loop that
may not stall on the device-wide synchronisation of cudaMalloc / cudaFree, a process whose
device memory was handed out in full at start-up).  The intermediate m = x A lives in a
fixed 1 MiB array inside the library image that every call shares, so the test calls it
twice in a row, with different batches, and checks both results against the ordinary entry
point, and checks that an oversized request is refused before anything runs.  This file
sorts last on purpose: a run that stops at the first failure has then run everything else.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2608_05483_b200 as P
from gpu_util import DEV, Runner
from helpers import TOL_FP32_PATH, random_problem

pytestmark = pytest.mark.gpu


def _both(r, p, ids_np):
    ids = torch.from_numpy(np.ascontiguousarray(ids_np, np.int32)).to(DEV)
    y_ref = torch.from_numpy(p["y_in"]).to(DEV)
    r.ctx.set_path(P.PATH_FUSED)
    r.ctx.bucket(ids, p["N"])
    r.ctx.lora_delta(r.x, ids, 0, 0, y_ref)
    y_new = torch.from_numpy(p["y_in"]).to(DEV)
    r.ctx.lora_delta_noalloc(r.x, ids, 0, 0, y_new)
    torch.cuda.synchronize()
    return y_new.cpu().numpy(), y_ref.cpu().numpy()


def test_two_calls_in_a_row_match_the_ordinary_entry_point():
    p = random_problem(4242, T=150, d_in=776, d_out=520, ranks=[8, 24, 64, 5, 16], with_minus_one=True)
    r = Runner(p)
    try:
        before = r.ctx.launch_count()
        ids_a = p["ids"]
        ids_b = np.roll(p["ids"], 17)           # second call: another batch over the same scratch array
        for ids in (ids_a, ids_b):
            got, ref = _both(r, p, ids)
            scale = np.max(np.abs(ref - p["y_in"]))
            assert np.max(np.abs(got - ref)) <= TOL_FP32_PATH * scale
            # and against the oracle, so that the two entry points cannot be wrong together
            want = oracle.lora_delta(p["x"], ids, p["ranks"], p["scales"], p["A"], p["B"], p["d_out"], p["y_in"])
            assert np.max(np.abs(got - want)) <= TOL_FP32_PATH * scale + 1e-6 * np.max(np.abs(want))
        assert r.ctx.launch_count() > before
        assert r.ctx.device_status() == 0
        # after the first call on the device (which looked the array's address up), a call allocates nothing:
        # the device's free memory is the same before and after, with everything the call needs made beforehand
        ids = torch.from_numpy(np.ascontiguousarray(ids_a, np.int32)).to(DEV)
        y = torch.from_numpy(p["y_in"]).to(DEV)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        rc = P.plora_lora_delta_noalloc(r.ctx.handle, r.x.data_ptr(), ids.data_ptr(), p["T"], 0, 0, y.data_ptr())
        torch.cuda.synchronize()
        assert rc == P.OK and torch.cuda.mem_get_info()[0] == free_before
    finally:
        r.close()


def test_request_beyond_the_fixed_array_is_refused():
    # padded maximum rank 128: the 1 MiB array holds 2048 tokens, not 2049
    p = random_problem(7, T=2049, d_in=64, d_out=64, ranks=[128, 8])
    r = Runner(p)
    try:
        y = torch.zeros((p["T"], 64), dtype=torch.float32, device=DEV)
        n0 = r.ctx.launch_count()
        rc = P.plora_lora_delta_noalloc(r.ctx.handle, r.x.data_ptr(), r.ids.data_ptr(), 2049, 0, 0, y.data_ptr())
        assert rc == P.ERR_WORKSPACE
        assert r.ctx.launch_count() == n0 and float(y.abs().max()) == 0.0
        rc = P.plora_lora_delta_noalloc(r.ctx.handle, r.x.data_ptr(), r.ids.data_ptr(), 2048, 0, 0, y.data_ptr())
        assert rc == P.OK
        torch.cuda.synchronize()
        want = oracle.lora_delta(p["x"][:2048], p["ids"][:2048], p["ranks"], p["scales"], p["A"], p["B"], 64)
        assert np.max(np.abs(y.cpu().numpy()[:2048] - want)) <= TOL_FP32_PATH * np.max(np.abs(want))
    finally:
        r.close()

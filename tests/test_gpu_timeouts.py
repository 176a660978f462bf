"""The give-up paths of the kernels' bounded waits, exercised without stalling the GPU.

A test hook makes one consumer of every CTA keep its stages, so the copy warp's wait for a free
stage runs out after a limit of a few milliseconds.  By then every copy the warp issued has landed
(the other consumers waited for them), so nothing is in flight when the kernel winds down.  Each
test checks the status word, that the rows around y were not written, that the status clears, and
that the next ordinary call on the same context (or workspace) is correct.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2608_05483_b200 as P
from gpu_util import DEV, Runner
from helpers import TOL_FP32_PATH, random_problem, rel_err

pytestmark = pytest.mark.gpu

LIMIT = 4_000_000   # SM clock cycles: about 2 ms, far below the hook's ceiling


def _guarded_y(T, d_out):
    buf = torch.full((T + 2, d_out), 777.0, dtype=torch.float32, device=DEV)
    buf[1:T + 1].zero_()
    return buf


def _tiny():
    # the Tiny shapes: 64 tokens, 512 -> 512, rank 8, 16 adapters
    return random_problem(11, T=64, d_in=512, d_out=512, ranks=[8] * 16, scales=[2.0] * 16)


def _small():
    # Small, but large enough that a CTA's copy warp goes round its ring of five stages: 160 one-token
    # segments at rank 16 over 4096 columns make about eight stages per CTA in every kernel (at the
    # Tiny shapes a CTA gets one stage and never waits for a free one, so the hook would not bite).
    p = random_problem(13, T=160, d_in=4096, d_out=4096, ranks=[16] * 160, scales=[2.0] * 160)
    p["ids"] = np.arange(160, dtype=np.int32)
    return p


def test_hook_needs_a_short_limit():
    r = Runner(_tiny())
    h = r.ctx.handle
    assert P.plora_set_test_hook(h, P.HOOK_WITHHOLD_RELEASE) == P.ERR_INVALID_ARG      # no limit set
    assert P.plora_set_wait_limit(h, P.HOOK_MAX_CYCLES + 1) == P.OK
    assert P.plora_set_test_hook(h, P.HOOK_WITHHOLD_RELEASE) == P.ERR_INVALID_ARG      # limit too long
    assert P.plora_set_wait_limit(h, -1) == P.ERR_INVALID_ARG
    assert P.plora_set_test_hook(h, 9) == P.ERR_INVALID_ARG
    assert P.plora_set_wait_limit(h, LIMIT) == P.OK
    assert P.plora_set_test_hook(h, P.HOOK_WITHHOLD_RELEASE) == P.OK
    assert P.plora_set_wait_limit(h, 0) == P.OK                                       # default limit drops the hook
    y = r.delta(P.PATH_FUSED)
    assert r.ctx.device_status() == 0 and np.any(y != 0)
    r.close()


@pytest.mark.parametrize("path", [P.PATH_FUSED, P.PATH_UNFUSED, P.PATH_SGMV, P.PATH_SGMV_SPLIT])
def test_a_wait_that_runs_out_is_reported_and_survivable(path):
    p = _small()
    r = Runner(p)
    ref = oracle.lora_delta(p["x"], p["ids"], p["ranks"], p["scales"], p["A"], p["B"], p["d_out"])
    r.ctx.set_path(path)
    r.ctx.set_wait_limit(LIMIT)
    r.ctx.set_test_hook(P.HOOK_WITHHOLD_RELEASE)
    buf = _guarded_y(p["T"], p["d_out"])
    r.ctx.bucket(r.ids, p["N"])
    r.ctx.lora_delta(r.x, r.ids, 0, 0, buf[1:p["T"] + 1])
    torch.cuda.synchronize()
    assert r.ctx.device_status() == P.ERR_TIMEOUT
    assert r.ctx.device_status() == 0                           # reading it cleared it
    out = buf.cpu().numpy()
    assert np.all(out[0] == 777.0) and np.all(out[-1] == 777.0), "rows around y were written"
    assert np.all(np.isfinite(out))
    # back to normal: same context, default limit, no hook
    r.ctx.set_test_hook(P.HOOK_NONE)
    r.ctx.set_wait_limit(0)
    for _ in range(2):
        got = r.delta(path)
        assert rel_err(got, ref) <= (5e-5 if path in (P.PATH_SGMV, P.PATH_SGMV_SPLIT) else TOL_FP32_PATH)
    assert r.ctx.device_status() == 0
    r.close()


def test_a_wait_that_runs_out_in_a_launch_that_joins_late():
    # the same with the inputs-resident hint: the consumers of the fused kernel have not joined the stream order
    # when the copy warp gives up; two calls in a row, so that the second starts under the first one's wind-down
    p = _small()
    r = Runner(p)
    ref = oracle.lora_delta(p["x"], p["ids"], p["ranks"], p["scales"], p["A"], p["B"], p["d_out"])
    r.ctx.set_path(P.PATH_FUSED)
    r.ctx.set_inputs_resident(True)
    r.ctx.set_wait_limit(LIMIT)
    r.ctx.set_test_hook(P.HOOK_WITHHOLD_RELEASE)
    buf = _guarded_y(p["T"], p["d_out"])
    r.ctx.bucket(r.ids, p["N"])
    r.ctx.lora_delta(r.x, r.ids, 0, 0, buf[1:p["T"] + 1])
    r.ctx.lora_delta(r.x, r.ids, 0, 0, buf[1:p["T"] + 1])
    torch.cuda.synchronize()
    assert r.ctx.device_status() == P.ERR_TIMEOUT
    out = buf.cpu().numpy()
    assert np.all(out[0] == 777.0) and np.all(out[-1] == 777.0), "rows around y were written"
    r.ctx.set_test_hook(P.HOOK_NONE)
    r.ctx.set_wait_limit(0)
    for _ in range(2):
        assert rel_err(r.delta(P.PATH_FUSED), ref) <= TOL_FP32_PATH
    assert r.ctx.device_status() == 0
    r.close()


def test_short_limit_alone_changes_nothing():
    p = random_problem(12, T=150, d_in=776, d_out=520, ranks=[8, 24, 64, 5, 16], with_minus_one=True)
    r = Runner(p)
    ref = oracle.lora_delta(p["x"], p["ids"], p["ranks"], p["scales"], p["A"], p["B"], p["d_out"])
    r.ctx.set_wait_limit(P.HOOK_MAX_CYCLES)
    for path in (P.PATH_FUSED, P.PATH_UNFUSED, P.PATH_SGMV, P.PATH_SGMV_SPLIT):
        assert rel_err(r.delta(path), ref) <= 1e-4
    assert r.ctx.device_status() == 0
    r.close()


@pytest.mark.parametrize("G", [1, 4])
def test_attention_wait_that_runs_out(G):
    from oracle.attention import decode_attention
    rng = np.random.default_rng(5 + G)
    n_req, H, L, d = 6, 2, 700, 128
    kv_len = rng.integers(300, L + 1, size=n_req).astype(np.int32)
    q = torch.from_numpy(rng.standard_normal((n_req, H * G, d), dtype=np.float32)).to(DEV).to(torch.bfloat16)
    K = torch.from_numpy(rng.standard_normal((n_req, H, L, d), dtype=np.float32)).to(DEV).to(torch.bfloat16)
    V = torch.from_numpy(rng.standard_normal((n_req, H, L, d), dtype=np.float32)).to(DEV).to(torch.bfloat16)
    lens = torch.from_numpy(kv_len).to(DEV)
    scale = 1.0 / np.sqrt(d)
    ws = torch.zeros(P.plora_attn_workspace_bytes(n_req, L, H, G), dtype=torch.uint8, device=DEV)
    assert P.plora_attn_set_debug(ws.data_ptr(), 0, P.HOOK_WITHHOLD_RELEASE) == P.ERR_INVALID_ARG
    assert P.plora_attn_set_debug(ws.data_ptr(), LIMIT, P.HOOK_WITHHOLD_RELEASE) == P.OK
    buf = torch.full((n_req + 2, H * G, d), 777.0, dtype=torch.float32, device=DEV)
    P.attn_decode(q, K, V, lens, scale, out=buf[1:n_req + 1], workspace=ws)
    torch.cuda.synchronize()
    rc, status = P.plora_attn_status(ws.data_ptr())
    assert rc == P.OK and status == P.ERR_TIMEOUT
    assert P.plora_attn_status(ws.data_ptr()) == (P.OK, 0)
    out = buf.cpu().numpy()
    assert np.all(out[0] == 777.0) and np.all(out[-1] == 777.0)
    assert P.plora_attn_set_debug(ws.data_ptr(), 0, P.HOOK_NONE) == P.OK
    got, _ = P.attn_decode(q, K, V, lens, scale, workspace=ws)
    torch.cuda.synchronize()
    ref = decode_attention(q.float().cpu().numpy().astype(np.float64), K.float().cpu().numpy().astype(np.float64),
                           V.float().cpu().numpy().astype(np.float64), kv_len, scale)
    assert np.max(np.abs(got.cpu().numpy() - ref)) <= 2e-5 * max(1.0, np.max(np.abs(ref)))
    assert P.plora_attn_status(ws.data_ptr()) == (P.OK, 0)

"""Full-size benchmark workloads, in the launch configuration bench.py times (AUTO path, one
layer of every config), checked on sampled output rows the oracle computes one by one.

Pools are drawn on the device (tens of GB would take minutes on the host); the adapters the
sampled tokens use are regenerated and copied back so the oracle sees the very same bits.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2608_05483_b200 as P
from bench import DeviceWorkload, algorithmic_bytes, bits_of
from helpers import TOL_CONTRACT, TOL_FP32_PATH
from workloads import make_workload

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("cfg", [2, 3, 4, 5, 6])
def test_sampled_rows_match_oracle(cfg):
    wl = make_workload(cfg, n_layers=1)
    dw = DeviceWorkload(wl, 0)
    try:
        dw.ctx.set_path(P.PATH_AUTO)
        y_in = {k: v.clone() for k, v in dw.y.items()}
        dw.step()
        torch.cuda.synchronize()
        assert dw.ctx.device_status() == 0
        # the bucket of the full batch, bit for bit
        got = dw.ctx.bucket_view()
        ref = oracle.bucket(wl.ids, wl.n_adapters)
        for k in ("perm", "seg_adapter", "seg_start"):
            assert got[k].tobytes() == ref[k].tobytes(), k
        assert got["n_seg"] == ref["n_seg"] and got["n_active"] == ref["n_active"]
        rng = np.random.default_rng(cfg)
        lens = np.bincount(wl.ids, minlength=wl.n_adapters)
        # sample tokens of the hottest adapter, of a one-token adapter and at random, first and last token included
        hot = np.flatnonzero(wl.ids == int(np.argmax(lens)))[:6]
        cold = np.flatnonzero(np.isin(wl.ids, np.flatnonzero(lens == lens[lens > 0].min())))[:6]
        sample = np.unique(np.concatenate([[0, wl.n_tok - 1], hot, cold, rng.integers(0, wl.n_tok, size=12)]))
        adapters = np.unique(wl.ids[sample])
        seen = set()
        for pool in wl.pools:
            if (pool.d_in, pool.d_out) in seen and pool.proj not in (0, 3):
                continue
            seen.add((pool.d_in, pool.d_out))
            A, B = dw.host_adapters(pool, adapters)
            x = bits_of(dw.x[(pool.layer, pool.x_group)])[sample]
            yi = y_in[(pool.layer, pool.proj)].cpu().numpy()[sample]
            want = oracle.lora_delta(x, wl.ids[sample], wl.ranks, wl.scales, A, B, pool.d_out, yi)
            have = dw.y[(pool.layer, pool.proj)].cpu().numpy()[sample]
            scale = np.max(np.abs(want - yi))
            err = np.max(np.abs(have - want))
            assert err <= TOL_CONTRACT * scale
            assert err <= TOL_FP32_PATH * scale + 1e-6 * np.max(np.abs(want)), (pool.name, err / scale)
    finally:
        dw.close()


def test_algorithmic_bytes_of_the_decode_config():
    wl = make_workload(2, n_layers=1)
    b = algorithmic_bytes(wl.ids, wl.ranks, 4096, 4096)
    assert b["adapter"] == b["distinct"] * (4096 + 4096) * 16 * 2
    assert b["x"] == 256 * 4096 * 2 and b["y"] == 256 * 4096 * 8


@pytest.mark.parametrize("cfg", [2, 3, 4, 5, 6])
def test_whole_output_of_one_projection_per_shape(cfg):
    """Every element of the [n_tok, d_out] output, for the first projection of each distinct shape, through the
    call the benchmark's step makes (q goes with its k and v), against the oracle at full size."""
    from bench import oracle_sample, parity_pools
    wl = make_workload(cfg, n_layers=1)
    dw = DeviceWorkload(wl, 0)
    try:
        dw.ctx.set_path(P.PATH_AUTO)
        pools, _, err, _, _ = oracle_sample(dw, 0, check_gpu=True, pools=parity_pools(wl))
        assert len(pools) == (3 if cfg == 3 else 1)
        assert err <= TOL_FP32_PATH, (cfg, err)
        assert dw.ctx.device_status() == 0
    finally:
        dw.close()

"""GPU LoRA delta vs the float64 oracle, element by element, through the C ABI.

Contract: max|gpu - ref| <= 5e-3 * max|ref| (bf16 inputs, fp32 accumulation).  The
BGMV paths keep m in fp32, so they are also held to 1e-4: an indexing mistake that
moves a few elements cannot hide under the contract's tolerance.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2608_05483_b200 as P
from gpu_util import DEV, Runner, bits_to_dev
from helpers import TOL_CONTRACT, TOL_FP32_PATH, random_problem, rel_err
from workloads.gen import f32_to_bf16_bits
from workloads import gen_adapter, gen_x, gen_y_in, make_workload

pytestmark = pytest.mark.gpu

BGMV_PATHS = [P.PATH_FUSED, P.PATH_UNFUSED]
# SGMV carries m as bf16 hi + lo (about 2^-17 relative), still far inside the fp32-path bound
ALL_PATHS = [P.PATH_FUSED, P.PATH_UNFUSED, P.PATH_SGMV, P.PATH_SGMV_SPLIT, P.PATH_AUTO]


def _oracle(p, y_in=None, ids=None):
    oracle.set_input_type(bool(p.get("fp16")))
    try:
        return oracle.lora_delta(p["x"], p["ids"] if ids is None else ids, p["ranks"], p["scales"], p["A"], p["B"],
                                 p["d_out"], y_in)
    finally:
        oracle.set_input_type(False)


def _problem_from_workload(wl, pool):
    AB = [gen_adapter(wl, pool, a) for a in range(wl.n_adapters)]
    return dict(T=wl.n_tok, d_in=pool.d_in, d_out=pool.d_out, N=wl.n_adapters, ranks=wl.ranks, scales=wl.scales,
                ids=wl.ids, x=gen_x(wl, pool), A=[ab[0] for ab in AB], B=[ab[1] for ab in AB],
                y_in=gen_y_in(wl, pool))


def _check_paths(p, paths=ALL_PATHS, tol=TOL_FP32_PATH, on_device=False):
    r = Runner(p, on_device=on_device)
    try:
        ref0 = _oracle(p)
        ref1 = _oracle(p, y_in=p["y_in"])
        for path in paths:
            got0 = r.delta(path)
            assert rel_err(got0, ref0) <= min(tol, TOL_CONTRACT), (path, rel_err(got0, ref0))
            got1 = r.delta(path, y_in=p["y_in"])
            # y_in enters with one fp32 rounding of the sum
            assert np.max(np.abs(got1 - ref1)) <= tol * np.max(np.abs(ref0)) + 1e-6 * np.max(np.abs(ref1)), path
            again = r.delta(path, y_in=p["y_in"])
            assert again.tobytes() == got1.tobytes(), "not bit-reproducible"
        assert r.ctx.device_status() == 0
    finally:
        r.close()


def test_tiny_config():
    wl = make_workload(1)
    _check_paths(_problem_from_workload(wl, wl.pools[0]))


def test_tiny_config_device_resident_sources():
    wl = make_workload(1)
    _check_paths(_problem_from_workload(wl, wl.pools[0]), on_device=True)


@pytest.mark.parametrize("cfg,kw", [
    (2, dict(n_adapters=200, d_model=1024, n_layers=1)),          # decode, Zipf ids, several tiles per matrix
    (3, dict(n_adapters=100, d_model=640, d_ff=1728, n_layers=1, n_tok=128)),   # rectangular projections, rank 64
    (4, dict(n_adapters=50, d_model=512, n_layers=1, n_tok=1024)),  # long contiguous segments
    (5, dict(n_adapters=60, d_model=1024, n_layers=1, n_tok=512)),  # mixed ranks, mixed segment lengths
    (5, dict(n_adapters=200, d_model=512, n_layers=1, n_tok=2048)),  # AUTO sends long segments to SGMV, short ones to BGMV
    (6, dict(n_adapters=120, d_model=1024, n_layers=1)),            # the paper's 80/50 skew, ranks 8..128
])
def test_reduced_benchmark_configs(cfg, kw):
    wl = make_workload(cfg, **kw)
    seen = set()
    for pool in wl.pools:
        if (pool.d_in, pool.d_out) in seen:
            continue
        seen.add((pool.d_in, pool.d_out))
        _check_paths(_problem_from_workload(wl, pool))


@pytest.mark.parametrize("r", [1, 2, 7, 8, 9, 16, 31, 33, 63, 64, 100, 128])
def test_odd_ranks(r):
    p = random_problem(100 + r, T=37, d_in=328, d_out=264, ranks=[r, max(1, r - 1), r], with_minus_one=True)
    _check_paths(p)


@pytest.mark.parametrize("d_in,d_out", [(8, 8), (64, 72), (520, 1032), (1048, 504), (2056, 4104)])
def test_ragged_dims(d_in, d_out):
    p = random_problem(d_in + d_out, T=19, d_in=d_in, d_out=d_out, ranks=[8, 16, 32, 64, 128, 4], with_minus_one=True)
    _check_paths(p)


@pytest.mark.parametrize("T", [1, 2, 3, 4, 5, 8, 9, 63, 257])
def test_token_counts_and_hot_adapter(T):
    p = random_problem(T, T=T, d_in=512, d_out=512, ranks=[16, 16, 8])
    p["ids"][: max(1, T // 2)] = 1      # one hot adapter: many units share its matrices
    _check_paths(p)


def test_auto_dispatch_uses_both_kernels():
    # 128 prefill runs of 64 tokens (>= 128 tensor-core tiles) followed by 300 single decode tokens
    rng = np.random.default_rng(21)
    N = 300
    ids = np.concatenate([np.repeat(rng.permutation(N)[:128], 64), rng.integers(0, N, size=300)]).astype(np.int32)
    p = random_problem(22, T=len(ids), d_in=256, d_out=320, ranks=rng.choice([8, 16, 32, 64], size=N))
    p["ids"] = ids
    lens = np.bincount(ids, minlength=N)
    assert (lens >= 64).sum() >= 128 and ((lens > 0) & (lens < 32)).any()
    r = Runner(p)
    try:
        r.ctx.set_path(P.PATH_AUTO)
        y = torch.zeros((p["T"], p["d_out"]), dtype=torch.float32, device=DEV)
        r.ctx.bucket(r.ids, p["N"])
        n0 = r.ctx.launch_count()
        r.ctx.lora_delta(r.x, r.ids, 0, 0, y)
        torch.cuda.synchronize()
        n_classes = len(set(int(v) for v in p["ranks"]))   # ranks 8..64 are their own padded classes
        # a large batch: the classify pass of a mixed-rank pool + one BGMV launch per rank class + the wide tensor-core launch
        assert r.ctx.launch_count() - n0 == 1 + n_classes + 1
        assert rel_err(y.cpu().numpy(), _oracle(p)) <= TOL_FP32_PATH
        # a decode-sized batch stays with BGMV
        small = torch.from_numpy(ids[-256:].copy()).to(DEV)
        y2 = torch.zeros((256, p["d_out"]), dtype=torch.float32, device=DEV)
        r.ctx.bucket(small, p["N"])
        n0 = r.ctx.launch_count()
        r.ctx.lora_delta(r.x[-256:], small, 0, 0, y2)
        torch.cuda.synchronize()
        assert r.ctx.launch_count() - n0 == 1 + 1     # classify + one launch for all classes
        assert rel_err(y2.cpu().numpy(), _oracle(p, ids=ids)[-256:]) <= TOL_FP32_PATH
        # few long segments in a batch too small for the wide shape: BGMV launches + the split tensor-core launch
        few = np.concatenate([np.repeat(np.arange(3), 200), rng.integers(0, N, size=500)]).astype(np.int32)
        few_t = torch.from_numpy(few).to(DEV)
        y3 = torch.zeros((len(few), p["d_out"]), dtype=torch.float32, device=DEV)
        r.ctx.bucket(few_t, p["N"])
        n0 = r.ctx.launch_count()
        r.ctx.lora_delta(r.x[:len(few)], few_t, 0, 0, y3)
        torch.cuda.synchronize()
        assert r.ctx.launch_count() - n0 == 1 + n_classes + 1    # classify + one BGMV launch per class (1100 rows) + split
        p3 = dict(p, x=p["x"][:len(few)], ids=few)
        assert rel_err(y3.cpu().numpy(), _oracle(p3)) <= TOL_FP32_PATH
    finally:
        r.close()


def _ids_from_runs(runs, shuffle_seed=None):
    """ids for consecutive runs [(adapter, length), ...]; optionally dealt out in a random order."""
    ids = np.concatenate([np.full(n, a, np.int32) for a, n in runs])
    if shuffle_seed is not None:
        np.random.default_rng(shuffle_seed).shuffle(ids)
    return ids


@pytest.mark.parametrize("layout", ["contiguous", "shuffled", "broken_runs"])
def test_sgmv_tile_shapes(layout):
    # segment lengths around the 64-row tile and the 32-row copy box: whole tiles, ragged last tiles,
    # a one-row tile, tokens that are consecutive (box copies), scattered (gather copies) or consecutive
    # in pieces that end inside a box
    lens = [128, 129, 33, 255, 300, 1, 31, 64, 65, 63]
    ranks = [8, 16, 32, 64, 128, 24, 5, 16, 32, 8]
    if layout == "broken_runs":
        runs = []
        for rep in range(3):      # every adapter's tokens come as three separate runs of uneven length
            runs += [(a, n // 3 + (rep == 2) * (n % 3)) for a, n in enumerate(lens)]
        ids = _ids_from_runs([r for r in runs if r[1] > 0])
    else:
        ids = _ids_from_runs(list(enumerate(lens)), shuffle_seed=5 if layout == "shuffled" else None)
    p = random_problem(300, T=len(ids), d_in=328, d_out=264, ranks=ranks)
    p["ids"] = ids
    _check_paths(p, paths=[P.PATH_SGMV, P.PATH_SGMV_SPLIT, P.PATH_AUTO])


@pytest.mark.parametrize("n_tok", [512, 2048])
def test_mixed_rank_calls_repeat_bit_for_bit(n_tok):
    # a small batch takes one launch for all rank classes; in a large one the class launches of a call
    # overlap and share the hand-over workspace and one epoch: a unit of one class must never see
    # another class's partial sums (a one-in-ten race when they met there)
    wl = make_workload(5, n_adapters=60, d_model=1024, n_layers=1, n_tok=n_tok)
    p = _problem_from_workload(wl, wl.pools[0])
    r = Runner(p)
    try:
        ref = _oracle(p, y_in=p["y_in"])
        first = r.delta(P.PATH_FUSED, y_in=p["y_in"])
        assert np.max(np.abs(first - ref)) <= TOL_FP32_PATH * np.max(np.abs(_oracle(p))) + 1e-6 * np.max(np.abs(ref))
        for _ in range(100):
            assert r.delta(P.PATH_FUSED, y_in=p["y_in"], guard=False).tobytes() == first.tobytes()
        assert r.ctx.device_status() == 0
    finally:
        r.close()


def test_cuda_graph_replay_of_a_mixed_call_sequence():
    # bucket + two dependent deltas (AUTO: classify, overlapping class launches, SGMV) captured once and
    # replayed: every replay must give the bits of the eager run
    rng = np.random.default_rng(31)
    N = 200
    ids = np.concatenate([np.repeat(rng.permutation(N)[:130], 64), rng.integers(0, N, size=300)]).astype(np.int32)
    p = random_problem(32, T=len(ids), d_in=256, d_out=320, ranks=rng.choice([8, 16, 32, 64, 128], size=N))
    p["ids"] = ids
    r = Runner(p)
    try:
        r.ctx.set_path(P.PATH_AUTO, sgmv_min_rows=32)
        y_in = torch.from_numpy(p["y_in"]).to(DEV)
        y = y_in.clone()

        def step():
            r.ctx.bucket(r.ids, p["N"])
            r.ctx.lora_delta(r.x, r.ids, 0, 0, y)       # y += delta(x)
            r.ctx.lora_delta(r.x, r.ids, 0, 0, y)       # and once more: depends on the first through y

        n0 = r.ctx.launch_count()
        step()
        torch.cuda.synchronize()
        assert r.ctx.launch_count() - n0 == 1 + (1 + 5 + 1) + (5 + 1)   # bucket; classify once; per delta: five classes, SGMV
        eager = y.cpu().numpy().copy()
        ref = _oracle(p)
        want = p["y_in"].astype(np.float64) + 2 * ref
        assert np.max(np.abs(eager - want)) <= TOL_FP32_PATH * np.max(np.abs(ref)) + 2e-6 * np.max(np.abs(want))
        s = torch.cuda.Stream()
        s.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(s):
            step()
        torch.cuda.current_stream().wait_stream(s)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            step()
        for _ in range(20):
            y.copy_(y_in)
            g.replay()
            torch.cuda.synchronize()
            assert y.cpu().numpy().tobytes() == eager.tobytes()
        assert r.ctx.device_status() == 0
    finally:
        r.close()


@pytest.mark.parametrize("seed", range(24))
def test_random_shapes_ranks_and_id_mixes(seed):
    # a sweep over what the kernels branch on: ragged dimensions, every rank class alone and mixed, ids that are
    # uniform, skewed, run-structured or mostly absent, batch sizes on both sides of the tensor-core threshold
    rng = np.random.default_rng(9000 + seed)
    d_in = int(rng.integers(1, 260)) * 8
    d_out = int(rng.integers(1, 260)) * 8
    N = int(rng.integers(1, 48))
    rank_sets = [[8], [16], [64], [128], [1, 2, 3], [8, 16, 32, 64, 128], [5, 33, 100], [16, 64]]
    ranks = rng.choice(rank_sets[seed % len(rank_sets)], size=N)
    T = int(rng.choice([1, 3, 17, 64, 200, 513, 700, 1500]))
    kind = seed % 4
    if kind == 0:
        ids = rng.integers(0, N, size=T)
    elif kind == 1:
        ids = np.minimum((rng.pareto(1.0, size=T)).astype(np.int64), N - 1)
    elif kind == 2:
        ids = np.repeat(rng.integers(0, N, size=T // 37 + 1), 37)[:T]
    else:
        ids = np.where(rng.random(T) < 0.7, -1, rng.integers(0, N, size=T))
    p = random_problem(9100 + seed, T=T, d_in=d_in, d_out=d_out, ranks=ranks, fp16=bool(seed & 8))
    p["ids"] = ids.astype(np.int32)
    _check_paths(p)


def test_empty_and_all_minus_one():
    p = random_problem(1, T=0, d_in=64, d_out=64, ranks=[8])
    r = Runner(p, max_tokens=8)
    assert r.delta(P.PATH_FUSED).shape == (0, 64)
    r.close()
    p = random_problem(2, T=9, d_in=64, d_out=64, ranks=[8, 8])
    p["ids"][:] = -1
    r = Runner(p)
    for path in ALL_PATHS:
        got = r.delta(path, y_in=p["y_in"])
        assert np.array_equal(got, p["y_in"])
    r.close()


def test_shrink_and_expand_entry_points():
    p = random_problem(77, T=45, d_in=776, d_out=520, ranks=[8, 24, 64, 5], with_minus_one=True)
    r = Runner(p)
    try:
        ldm = r.ctx.pool_max_rank(0, 0)
        assert ldm == 64
        m = torch.full((p["T"], ldm), 7.0, dtype=torch.float32, device=DEV)
        r.ctx.shrink(r.x, r.ids, 0, 0, m)
        torch.cuda.synchronize()
        m_ref = oracle.shrink(p["x"], p["ids"], p["ranks"], p["A"], ldm=ldm)
        assert rel_err(m.cpu().numpy(), m_ref) <= TOL_FP32_PATH
        assert np.all(m.cpu().numpy()[m_ref == 0] == 0)      # padding columns and id -1 rows are exact zeros
        y = torch.from_numpy(p["y_in"]).to(DEV)
        r.ctx.expand(m, r.ids, 0, 0, y)
        torch.cuda.synchronize()
        y_ref = oracle.expand(m.cpu().numpy().astype(np.float64), p["ids"], p["ranks"], p["scales"], p["B"], p["d_out"],
                              p["y_in"])
        delta_scale = np.max(np.abs(y_ref - p["y_in"]))
        assert np.max(np.abs(y.cpu().numpy() - y_ref)) <= TOL_FP32_PATH * delta_scale + 1e-6 * np.max(np.abs(y_ref))
    finally:
        r.close()


def test_out_of_range_id_is_skipped_and_flagged():
    p = random_problem(5, T=12, d_in=256, d_out=256, ranks=[8, 16])
    ids = p["ids"].copy()
    ids[4] = 2          # == n_adapters
    r = Runner(p)
    got = r.delta(P.PATH_FUSED, y_in=p["y_in"], ids=ids)
    assert r.ctx.device_status() == P.ERR_BAD_ADAPTER_ID
    ids_ref = ids.copy(); ids_ref[4] = -1
    ref = _oracle(p, y_in=p["y_in"], ids=ids_ref)
    assert np.array_equal(got[4], p["y_in"][4])
    assert np.max(np.abs(got - ref)) <= 1e-4 * np.max(np.abs(ref))
    r.close()


@pytest.mark.parametrize("case", ["decode", "ragged", "segments"])
def test_half_precision_inputs(case):
    # the paper's own FP16: x, A and B as IEEE half; every path, the same bounds as for bf16
    if case == "decode":
        p = random_problem(501, T=61, d_in=1024, d_out=768, ranks=[16, 16, 8, 64, 128, 3], with_minus_one=True, fp16=True)
    elif case == "ragged":
        p = random_problem(502, T=19, d_in=520, d_out=1032, ranks=[8, 16, 32, 64, 128, 4], with_minus_one=True, fp16=True)
    else:
        p = random_problem(503, T=700, d_in=328, d_out=264, ranks=[8, 16, 32, 64, 128, 24], fp16=True)
        p["ids"] = _ids_from_runs([(0, 129), (1, 64), (2, 255), (3, 33), (4, 130), (5, 89)])
    _check_paths(p)


def test_two_byte_m_between_shrink_and_expand():
    # the paper's strategy E4 ships m at 2 bytes per value: shrink rounds the fp32 sum to bf16, expand widens it again
    from workloads import bf16_bits_to_f64, f32_to_bf16_bits
    p = random_problem(78, T=53, d_in=776, d_out=520, ranks=[8, 24, 64, 5, 128], with_minus_one=True)
    r = Runner(p)
    try:
        ldm = r.ctx.pool_max_rank(0, 0)
        assert ldm == 128
        m16 = torch.full((p["T"], ldm), 7.0, dtype=torch.bfloat16, device=DEV)
        r.ctx.shrink_m16(r.x, r.ids, 0, 0, m16)
        torch.cuda.synchronize()
        got_bits = m16.view(torch.int16).cpu().numpy().view(np.uint16)
        m_ref = oracle.shrink(p["x"], p["ids"], p["ranks"], p["A"], ldm=ldm)
        want_bits = f32_to_bf16_bits(m_ref.astype(np.float32))
        # the same value rounded from an fp32 sum (device) or from the float64 sum (oracle) may fall on either side
        # of a rounding boundary: at most one bf16 step apart, and only rarely
        step = np.abs(got_bits.astype(np.int32) - want_bits.astype(np.int32))
        assert step.max() <= 1 and (step > 0).mean() < 0.01
        assert np.all(got_bits[m_ref == 0] == 0)       # padding columns and id -1 rows are exact zeros
        # expand from a given 2-byte m: no rounding decision left, the fp32-path bound applies
        m_in = torch.from_numpy(want_bits.view(np.int16)).to(DEV).view(torch.bfloat16)
        y = torch.from_numpy(p["y_in"]).to(DEV)
        r.ctx.expand_m16(m_in, r.ids, 0, 0, y)
        torch.cuda.synchronize()
        ref = oracle.expand(bf16_bits_to_f64(want_bits), p["ids"], p["ranks"], p["scales"], p["B"], p["d_out"], p["y_in"])
        delta = oracle.lora_delta(p["x"], p["ids"], p["ranks"], p["scales"], p["A"], p["B"], p["d_out"], None)
        assert np.max(np.abs(y.cpu().numpy() - ref)) <= TOL_FP32_PATH * np.max(np.abs(delta)) + 1e-6 * np.max(np.abs(ref))
        # the pair against the unrounded definition: inside the contract, with the cost of one bf16 rounding
        y2 = torch.zeros((p["T"], p["d_out"]), dtype=torch.float32, device=DEV)
        r.ctx.expand_m16(m16, r.ids, 0, 0, y2)
        torch.cuda.synchronize()
        err = rel_err(y2.cpu().numpy(), delta)
        assert 1e-5 < err <= TOL_CONTRACT
        # ldm must keep the rows of m 16-byte aligned
        bad = torch.zeros((p["T"], ldm + 4), dtype=torch.bfloat16, device=DEV)
        with pytest.raises(P.PloraError):
            r.ctx.shrink_m16(r.x, r.ids, 0, 0, bad)
        assert r.ctx.device_status() == 0
    finally:
        r.close()


@pytest.mark.parametrize("rank", [40, 64, 100, 128])
@pytest.mark.parametrize("n_distinct", [3, 30, 140])
def test_high_rank_units_few_and_many(rank, n_distinct):
    # a launch with few units of padded rank 64 or 128 cuts their shrink into row slices, one with
    # many units does not (the launch decides from its unit count); the widths are ragged against
    # both geometries (64 and 256 columns per stage) and units have 1..4 tokens
    rng = np.random.default_rng(rank * 1000 + n_distinct)
    N = n_distinct + 5
    p = random_problem(rank + n_distinct, T=1, d_in=584, d_out=328, ranks=[rank] * N)
    ids = np.concatenate([np.repeat(np.arange(n_distinct), 1), rng.integers(0, n_distinct, n_distinct // 2 + 2)]).astype(np.int32)
    rng.shuffle(ids)
    T = len(ids)
    p["T"], p["ids"] = T, ids
    p["x"] = f32_to_bf16_bits(rng.standard_normal((T, p["d_in"]), dtype=np.float32))
    p["y_in"] = rng.standard_normal((T, p["d_out"]), dtype=np.float32)
    _check_paths(p, paths=(P.PATH_FUSED, P.PATH_AUTO))


def test_widest_projection_highest_and_lowest_rank_largest_batch_per_adapter():
    # the corners of the paper's parameter ranges (Section V-A: D up to 16384, R from 2 to 128, up to 256
    # requests on one adapter) in one batch
    ranks = [128, 2, 64, 3, 128, 17]
    rng = np.random.default_rng(404)
    ids = np.concatenate([np.full(256, 0), np.full(40, 1), rng.integers(2, 6, size=60), np.full(3, -1)]).astype(np.int32)
    rng.shuffle(ids)
    p = random_problem(405, T=len(ids), d_in=16384, d_out=16384, ranks=ranks)
    p["ids"] = ids
    _check_paths(p, paths=(P.PATH_FUSED, P.PATH_UNFUSED, P.PATH_SGMV, P.PATH_SGMV_SPLIT, P.PATH_AUTO))


def test_host_buffer_entry_point():
    p = random_problem(6, T=33, d_in=512, d_out=384, ranks=[16, 8, 32])
    r = Runner(p, max_tokens=64)
    r.ctx.set_path(P.PATH_FUSED)
    x_h = torch.from_numpy(p["x"].view(np.int16)).pin_memory()
    ids_h = torch.from_numpy(p["ids"]).pin_memory()
    y_h = torch.from_numpy(p["y_in"].copy()).pin_memory()
    r.ctx.lora_delta_host(x_h, ids_h, 0, 0, y_h)
    ref = _oracle(p, y_in=p["y_in"])
    assert np.max(np.abs(y_h.numpy() - ref)) <= 1e-4 * np.max(np.abs(ref))
    # numpy (pageable) buffers work too
    y_np = p["y_in"].copy()
    r.ctx.lora_delta_host(p["x"], p["ids"], 0, 0, y_np)
    assert y_np.tobytes() == y_h.numpy().tobytes()
    r.close()


def test_pipelined_host_calls_overlap_and_keep_every_result():
    # more queued calls than staging sets, each with its own ids, x and y; q/k/v share one x and go
    # as one call, o goes alone; every result equals the device-buffer path bit for bit
    wl = make_workload(2, n_adapters=48, d_model=512, n_layers=1, n_tok=120)
    ctx = P.Context(wl.n_tok, wl.n_adapters)
    probs = {}
    for pool in wl.pools:
        pr = _problem_from_workload(wl, pool)
        probs[pool.proj] = pr
        ctx.register_pool(pool.layer, pool.proj, pool.d_in, pool.d_out, wl.ranks, wl.scales, pr["A"], pr["B"])
    ctx.set_path(P.PATH_AUTO)
    rng = np.random.default_rng(5)
    calls = []
    for i in range(9):
        n_tok = int(rng.integers(1, wl.n_tok + 1))
        ids = rng.integers(-1, wl.n_adapters, n_tok).astype(np.int32)
        projs = [0, 1, 2] if i % 2 == 0 else [3]
        x = probs[projs[0]]["x"][:n_tok].copy()
        x[:, :8] = x[::-1, :8]                      # a different x per call
        ys = [rng.standard_normal((n_tok, probs[pj]["d_out"])).astype(np.float32) for pj in projs]
        calls.append(dict(ids=ids, projs=projs, x=x, y_in=[y.copy() for y in ys],
                          x_h=torch.from_numpy(x.view(np.int16)).pin_memory(), ids_h=torch.from_numpy(ids).pin_memory(),
                          y_h=[torch.from_numpy(y).pin_memory() for y in ys]))
    for c in calls:
        ctx.lora_delta_host_async(c["x_h"], c["ids_h"], [0] * len(c["projs"]), c["projs"], c["y_h"])
    ctx.host_sync()
    for c in calls:
        ids_d = torch.from_numpy(c["ids"]).to(DEV)
        x_d = bits_to_dev(c["x"])
        for g, pj in enumerate(c["projs"]):
            y_d = torch.from_numpy(c["y_in"][g]).to(DEV)
            ctx.lora_delta(x_d, ids_d, 0, pj, y_d)
            torch.cuda.synchronize()
            assert c["y_h"][g].numpy().tobytes() == y_d.cpu().numpy().tobytes(), (c["projs"], g)
            pr = dict(probs[pj], T=len(c["ids"]), ids=c["ids"], x=c["x"])
            ref = _oracle(pr, y_in=c["y_in"][g])
            delta = np.max(np.abs(ref - c["y_in"][g]))
            assert np.max(np.abs(c["y_h"][g].numpy() - ref)) <= TOL_FP32_PATH * delta + 1e-6 * np.max(np.abs(ref))
    assert ctx.device_status() == 0
    # one x cannot serve pools of different input width; unknown pools are refused
    assert P.plora_lora_delta_host_async(ctx.handle, 0, 0, 0, [0], [9], [0]) == P.ERR_NOT_REGISTERED
    c = calls[0]
    assert P.plora_lora_delta_host_async(ctx.handle, c["x_h"].data_ptr(), c["ids_h"].data_ptr(), len(c["ids"]), [0] * 5,
                                         [0] * 5, [c["y_h"][0].data_ptr()] * 5) == P.ERR_INVALID_ARG
    ctx.close()


def test_pools_with_different_ranks_share_a_bucket():
    # the sort of a batch's units by rank class is kept between calls and redone when a call's pool
    # has other ranks than the pool it was made for
    rng = np.random.default_rng(77)
    N, T = 40, 150
    ranks_a = rng.choice([8, 16, 64, 128], size=N)
    ranks_b = rng.choice([8, 32, 64], size=N)
    pa = random_problem(78, T=T, d_in=320, d_out=200, ranks=ranks_a)
    pb = random_problem(79, T=T, d_in=320, d_out=200, ranks=ranks_b)
    pb["ids"] = pa["ids"]
    pb["x"], pb["xf"] = pa["x"], pa["xf"]
    ctx = P.Context(T, N)
    ctx.register_pool(0, 0, 320, 200, pa["ranks"], pa["scales"], pa["A"], pa["B"])
    ctx.register_pool(0, 1, 320, 200, pb["ranks"], pb["scales"], pb["A"], pb["B"])
    ctx.register_pool(1, 0, 320, 200, pa["ranks"], pa["scales"], pa["A"], pa["B"])
    ctx.set_path(P.PATH_FUSED)
    ids = torch.from_numpy(pa["ids"]).to(DEV)
    x = bits_to_dev(pa["x"])
    ctx.bucket(ids, N)
    ref = {0: _oracle(pa), 1: _oracle(pb)}
    n0 = ctx.launch_count()
    order = [(0, 0), (1, 0), (0, 1), (0, 1), (0, 0), (1, 0)]   # same ranks, same, other, same, other, same
    for layer, proj in order:
        y = torch.zeros((T, 200), dtype=torch.float32, device=DEV)
        ctx.lora_delta(x, ids, layer, proj, y)
        torch.cuda.synchronize()
        assert rel_err(y.cpu().numpy(), ref[proj]) <= TOL_FP32_PATH, (layer, proj)
    assert ctx.launch_count() - n0 == len(order) + 3   # three sorts: at the start and at the two changes
    # a group whose pools have different ranks runs one projection after the other
    ya = torch.zeros((T, 200), dtype=torch.float32, device=DEV)
    yb = torch.zeros((T, 200), dtype=torch.float32, device=DEV)
    ctx.lora_delta_group([x, x], ids, [0, 0], [0, 1], [ya, yb])
    torch.cuda.synchronize()
    assert rel_err(ya.cpu().numpy(), ref[0]) <= TOL_FP32_PATH and rel_err(yb.cpu().numpy(), ref[1]) <= TOL_FP32_PATH
    assert ctx.device_status() == 0
    ctx.close()


def test_grouped_projections_of_a_mixed_rank_pool():
    # q, k, v with ranks from every class in one all-classes launch (small batch): bit-identical to three
    # separate calls, repeatable, and equal to the oracle
    rng = np.random.default_rng(611)
    N, T, d = 30, 90, 264
    ranks = rng.choice([4, 8, 16, 32, 64, 128], size=N)
    probs = [random_problem(612 + j, T=T, d_in=d, d_out=d, ranks=ranks) for j in range(3)]
    for pr in probs[1:]:
        pr["ids"], pr["x"], pr["xf"] = probs[0]["ids"], probs[0]["x"], probs[0]["xf"]
    ctx = P.Context(T, N)
    for j, pr in enumerate(probs):
        ctx.register_pool(0, j, d, d, pr["ranks"], pr["scales"], pr["A"], pr["B"])
    ctx.set_path(P.PATH_AUTO)
    ids = torch.from_numpy(probs[0]["ids"]).to(DEV)
    x = bits_to_dev(probs[0]["x"])
    ctx.bucket(ids, N)
    sep = []
    for j in range(3):
        y = torch.from_numpy(probs[j]["y_in"]).to(DEV)
        ctx.lora_delta(x, ids, 0, j, y)
        sep.append(y)
    torch.cuda.synchronize()
    for rep in range(20):
        ys = [torch.from_numpy(probs[j]["y_in"]).to(DEV) for j in range(3)]
        n0 = ctx.launch_count()
        ctx.lora_delta_group([x, x, x], ids, [0, 0, 0], [0, 1, 2], ys)
        torch.cuda.synchronize()
        assert ctx.launch_count() - n0 == 1      # the sort by rank class is kept from the first call
        for j in range(3):
            assert ys[j].cpu().numpy().tobytes() == sep[j].cpu().numpy().tobytes(), (rep, j)
    for j in range(3):
        ref = _oracle(probs[j], y_in=probs[j]["y_in"])
        delta = np.max(np.abs(ref - probs[j]["y_in"]))
        assert np.max(np.abs(sep[j].cpu().numpy() - ref)) <= TOL_FP32_PATH * delta + 1e-6 * np.max(np.abs(ref))
    assert ctx.device_status() == 0
    ctx.close()


def test_grouped_projections_share_a_launch():
    # q, k, v of one layer read the same x; o has its own.  Grouped q/k/v = one launch, bit-identical
    # to three separate calls (every y element still receives exactly one addition).
    wl = make_workload(2, n_adapters=64, d_model=768, n_layers=1, n_tok=200)
    ctx = P.Context(wl.n_tok, wl.n_adapters)
    ids = torch.from_numpy(wl.ids).to(DEV)
    probs = {}
    for pool in wl.pools:
        pr = _problem_from_workload(wl, pool)
        probs[pool.proj] = pr
        ctx.register_pool(pool.layer, pool.proj, pool.d_in, pool.d_out, wl.ranks, wl.scales, pr["A"], pr["B"])
    ctx.set_path(P.PATH_AUTO)
    ctx.bucket(ids, wl.n_adapters)
    x_qkv = bits_to_dev(probs[0]["x"])
    x_o = bits_to_dev(probs[3]["x"])
    y_sep = {}
    for proj in (0, 1, 2, 3):
        y_sep[proj] = torch.from_numpy(probs[proj]["y_in"]).to(DEV)
        ctx.lora_delta(x_qkv if proj < 3 else x_o, ids, 0, proj, y_sep[proj])
    y_grp = {proj: torch.from_numpy(probs[proj]["y_in"]).to(DEV) for proj in (0, 1, 2, 3)}
    n0 = ctx.launch_count()
    ctx.lora_delta_group([x_qkv, x_qkv, x_qkv], ids, [0, 0, 0], [0, 1, 2], [y_grp[0], y_grp[1], y_grp[2]])
    assert ctx.launch_count() - n0 == 1
    ctx.lora_delta_group([x_o], ids, [0], [3], [y_grp[3]])
    torch.cuda.synchronize()
    for proj in (0, 1, 2, 3):
        assert y_grp[proj].cpu().numpy().tobytes() == y_sep[proj].cpu().numpy().tobytes(), proj
        ref = _oracle(probs[proj], y_in=probs[proj]["y_in"])
        delta = np.max(np.abs(ref - probs[proj]["y_in"]))
        assert np.max(np.abs(y_grp[proj].cpu().numpy() - ref)) <= TOL_FP32_PATH * delta + 1e-6 * np.max(np.abs(ref))
    assert ctx.device_status() == 0
    # pools of different shape fall back to one launch each; bad arguments are refused
    assert P.plora_lora_delta_group(ctx.handle, [x_qkv.data_ptr()] * 5, ids.data_ptr(), wl.n_tok, [0] * 5, [0] * 5,
                                    [y_grp[0].data_ptr()] * 5) == P.ERR_INVALID_ARG
    assert P.plora_lora_delta_group(ctx.handle, [x_qkv.data_ptr()], ids.data_ptr(), wl.n_tok, [7], [0],
                                    [y_grp[0].data_ptr()]) == P.ERR_NOT_REGISTERED
    ctx.close()


def test_two_pools_and_bucket_reuse():
    wl = make_workload(2, n_adapters=64, d_model=512, n_layers=2, n_tok=96)
    ctx = P.Context(wl.n_tok, wl.n_adapters)
    ids = torch.from_numpy(wl.ids).to(DEV)
    probs = {}
    for pool in wl.pools:
        pr = _problem_from_workload(wl, pool)
        probs[(pool.layer, pool.proj)] = pr
        ctx.register_pool(pool.layer, pool.proj, pool.d_in, pool.d_out, wl.ranks, wl.scales, pr["A"], pr["B"])
    ctx.set_path(P.PATH_FUSED)
    ctx.bucket(ids, wl.n_adapters)
    before = ctx.launch_count()
    ys = {}
    for key, pr in probs.items():
        y = torch.zeros((wl.n_tok, pr["d_out"]), dtype=torch.float32, device=DEV)
        ctx.lora_delta(bits_to_dev(pr["x"]), ids, key[0], key[1], y)
        ys[key] = y
    torch.cuda.synchronize()
    assert ctx.launch_count() - before == len(probs)    # one kernel per call, the bucket is reused
    for key, pr in probs.items():
        assert rel_err(ys[key].cpu().numpy(), _oracle(pr)) <= TOL_FP32_PATH
    ctx.close()


def test_ids_rewritten_in_place_between_calls_without_plora_bucket():
    """A serving loop that refills one ids buffer every step and never calls plora_bucket: every call must
    bucket the ids it is given (a bucket made inside a delta call serves that call only), while a bucket made
    by plora_bucket is reused until the next plora_bucket."""
    p = random_problem(77, T=96, d_in=256, d_out=264, ranks=[8, 16, 32, 64, 8, 16], with_minus_one=True)
    r = Runner(p)
    try:
        ids_dev = r.ids.clone()
        rng = np.random.default_rng(1)
        for path in (P.PATH_FUSED, P.PATH_UNFUSED, P.PATH_AUTO):
            r.ctx.set_path(path)
            for step in range(3):
                ids = rng.integers(-1, p["N"], size=p["T"]).astype(np.int32)
                ids_dev.copy_(torch.from_numpy(ids))            # same address, new contents, no plora_bucket
                y = torch.from_numpy(p["y_in"]).to(DEV)
                n0 = r.ctx.launch_count()
                r.ctx.lora_delta(r.x, ids_dev, 0, 0, y)
                torch.cuda.synchronize()
                assert r.ctx.launch_count() - n0 >= 2           # the bucket kernel ran again
                want = oracle.lora_delta(p["x"], ids, p["ranks"], p["scales"], p["A"], p["B"], p["d_out"], p["y_in"])
                scale = np.max(np.abs(want - p["y_in"]))
                assert np.max(np.abs(y.cpu().numpy() - want)) <= TOL_FP32_PATH * scale + 1e-6 * np.max(np.abs(want)), (path, step)
        # an explicit bucket is reused: the second call launches no bucket kernel
        r.ctx.set_path(P.PATH_FUSED)
        r.ctx.bucket(ids_dev, p["N"])
        y = torch.zeros((p["T"], p["d_out"]), dtype=torch.float32, device=DEV)
        r.ctx.lora_delta(r.x, ids_dev, 0, 0, y)
        n0 = r.ctx.launch_count()
        r.ctx.lora_delta(r.x, ids_dev, 0, 0, y)
        per_call = r.ctx.launch_count() - n0
        r.ctx.lora_delta(r.x, ids_dev.clone(), 0, 0, y)         # other buffer: buckets again
        assert r.ctx.launch_count() - n0 - per_call >= per_call + 1   # + the bucket kernel (and the rank sort)
        assert r.ctx.device_status() == 0
    finally:
        r.close()


def test_three_long_segments_in_a_decode_batch_take_the_tensor_cores():
    """2048 tokens: three segments of 200 tokens among 1448 one- and two-token segments (the paper's per-adapter
    batches range up to 256 inside one step).  The long segments make ten tiles, far too few for a CTA per tile:
    AUTO sends them to the split tensor-core launch (a cluster per tile) and the rest to BGMV."""
    rng = np.random.default_rng(31)
    N = 900
    ids = np.concatenate([np.repeat(np.array([5, 17, 333]), 200), rng.integers(0, N, size=1448)]).astype(np.int32)
    rng.shuffle(ids)
    p = random_problem(32, T=2048, d_in=1024, d_out=1032, ranks=np.full(N, 16))
    p["ids"] = ids
    r = Runner(p)
    try:
        ref = _oracle(p)
        outs = {}
        for path in (P.PATH_AUTO, P.PATH_FUSED):
            r.ctx.set_path(path)
            y = torch.zeros((p["T"], p["d_out"]), dtype=torch.float32, device=DEV)
            r.ctx.bucket(r.ids, p["N"])
            n0 = r.ctx.launch_count()
            r.ctx.lora_delta(r.x, r.ids, 0, 0, y)
            torch.cuda.synchronize()
            n = r.ctx.launch_count() - n0
            assert n == (2 if path == P.PATH_AUTO else 1)      # one BGMV launch (one rank class) + the tensor-core launch
            outs[path] = y.cpu().numpy()
            assert rel_err(outs[path], ref) <= TOL_FP32_PATH, path
        # the long segments' rows came from another kernel: m went through its hi + lo split there
        long_rows = np.isin(ids, [5, 17, 333])
        assert not np.array_equal(outs[P.PATH_AUTO][long_rows], outs[P.PATH_FUSED][long_rows])
        assert r.ctx.device_status() == 0
    finally:
        r.close()


def test_grouped_call_with_long_segments_in_a_mid_sized_batch():
    """q, k, v of a layer in one call on a 1536-token batch with a few long segments: the three split tensor-core
    launches go ahead of the one BGMV launch of the group; results as from three separate calls, and as the oracle's."""
    rng = np.random.default_rng(41)
    N = 400
    ids = np.concatenate([np.repeat(np.array([3, 77]), 150), rng.integers(-1, N, size=1236)]).astype(np.int32)
    rng.shuffle(ids)
    p = random_problem(42, T=len(ids), d_in=512, d_out=520, ranks=np.full(N, 32))
    p["ids"] = ids
    ctx = P.Context(p["T"], N)
    try:
        xd = bits_to_dev(p["x"])
        idt = torch.from_numpy(ids).to(DEV)
        Bs = []
        for proj in range(3):
            B = [f32_to_bf16_bits(np.random.default_rng(100 + proj).standard_normal(b.shape, dtype=np.float32) / np.float32(np.sqrt(32))) for b in p["B"]]
            Bs.append(B)
            ctx.register_pool(0, proj, p["d_in"], p["d_out"], p["ranks"], p["scales"], p["A"], B)
        ctx.set_path(P.PATH_AUTO)
        ys = [torch.zeros((p["T"], p["d_out"]), dtype=torch.float32, device=DEV) for _ in range(3)]
        ctx.bucket(idt, N)
        n0 = ctx.launch_count()
        ctx.lora_delta_group([xd] * 3, idt, [0] * 3, [0, 1, 2], ys)
        torch.cuda.synchronize()
        assert ctx.launch_count() - n0 == 3 + 1            # three split launches, one BGMV launch for the group
        for proj in range(3):
            want = oracle.lora_delta(p["x"], ids, p["ranks"], p["scales"], p["A"], Bs[proj], p["d_out"])
            assert rel_err(ys[proj].cpu().numpy(), want) <= TOL_FP32_PATH, proj
            alone = torch.zeros_like(ys[proj])
            ctx.lora_delta(xd, idt, 0, proj, alone)
            torch.cuda.synchronize()
            assert rel_err(alone.cpu().numpy(), want) <= TOL_FP32_PATH
        assert ctx.device_status() == 0
    finally:
        ctx.close()


@pytest.mark.parametrize("rank", [8, 32])
def test_grouped_call_on_a_prefill_batch(rank):
    """q, k, v of a layer on a batch whose long segments all go to the wide tensor-core shape: one BGMV launch for the
    group's short segments and one tensor-core launch per projection (their own A, B and scales); results as the
    oracle's, and as from separate calls."""
    rng = np.random.default_rng(51)
    N, n_seg = 200, 130
    ids = np.concatenate([np.repeat(rng.permutation(N)[:n_seg], 64), rng.integers(-1, N, size=180)]).astype(np.int32)
    p = random_problem(52 + rank, T=len(ids), d_in=328, d_out=264, ranks=np.full(N, rank))
    p["ids"] = ids
    ctx = P.Context(p["T"], N)
    try:
        xd = bits_to_dev(p["x"])
        idt = torch.from_numpy(ids).to(DEV)
        pools = []
        for proj in range(3):
            r2 = np.random.default_rng(200 + proj)
            A = [f32_to_bf16_bits(r2.standard_normal(a.shape, dtype=np.float32) / np.float32(np.sqrt(p["d_in"]))) for a in p["A"]]
            B = [f32_to_bf16_bits(r2.standard_normal(b.shape, dtype=np.float32) / np.float32(np.sqrt(rank))) for b in p["B"]]
            sc = r2.choice(np.array([0.5, 1.0, 2.0], np.float32), size=N).astype(np.float32)
            pools.append((A, B, sc))
            ctx.register_pool(0, proj, p["d_in"], p["d_out"], p["ranks"], sc, A, B)
        ctx.set_path(P.PATH_AUTO)
        ys = [torch.from_numpy(p["y_in"]).to(DEV) for _ in range(3)]
        ctx.bucket(idt, N)
        n0 = ctx.launch_count()
        ctx.lora_delta_group([xd] * 3, idt, [0] * 3, [0, 1, 2], ys)
        torch.cuda.synchronize()
        assert ctx.launch_count() - n0 == 1 + 3            # one BGMV launch for the group, one tensor-core launch per projection
        for proj, (A, B, sc) in enumerate(pools):
            want = oracle.lora_delta(p["x"], ids, p["ranks"], sc, A, B, p["d_out"], p["y_in"])
            scale = np.max(np.abs(want - p["y_in"]))
            got = ys[proj].cpu().numpy()
            assert np.max(np.abs(got - want)) <= TOL_FP32_PATH * scale + 1e-6 * np.max(np.abs(want)), proj
            alone = torch.from_numpy(p["y_in"]).to(DEV)
            ctx.lora_delta(xd, idt, 0, proj, alone)
            torch.cuda.synchronize()
            assert np.max(np.abs(alone.cpu().numpy() - want)) <= TOL_FP32_PATH * scale + 1e-6 * np.max(np.abs(want))
        assert ctx.device_status() == 0
    finally:
        ctx.close()


@pytest.mark.parametrize("ranks, T, dims", [
    ([16] * 40, 96, (1024, 768)),                      # one rank class: the one-rank kernel
    ([8, 16, 32, 64, 128, 24] * 6, 120, (776, 520)),   # a small batch on a pool of mixed ranks: one launch for all classes
    ([8, 16, 32, 64] * 10, 1400, (256, 320)),          # a large batch on mixed ranks: one launch per class, overlapping
])
def test_inputs_resident_hint_changes_nothing_in_the_result(ranks, T, dims):
    # With the hint the fused kernels read x and start multiplying before the previous kernel of the stream has
    # ended; they write only after it has.  A chain of back-to-back deltas into one y (each depends on the one
    # before through y) must give the same bits with and without the hint, eagerly and from a CUDA graph.
    p = random_problem(900 + T, T=T, d_in=dims[0], d_out=dims[1], ranks=ranks, with_minus_one=True)
    r = Runner(p)
    try:
        r.ctx.set_path(P.PATH_FUSED)
        y_in = torch.from_numpy(p["y_in"]).to(DEV)
        y = y_in.clone()

        def step():
            r.ctx.bucket(r.ids, p["N"])
            for _ in range(4):
                r.ctx.lora_delta(r.x, r.ids, 0, 0, y)

        results = {}
        for hint in (False, True, False):
            r.ctx.set_inputs_resident(hint)
            y.copy_(y_in)
            step()
            torch.cuda.synchronize()
            results.setdefault(hint, []).append(y.cpu().numpy().copy())
        ref = _oracle(p)
        want = p["y_in"].astype(np.float64) + 4 * ref
        assert np.max(np.abs(results[True][0] - want)) <= TOL_FP32_PATH * np.max(np.abs(ref)) + 4e-6 * np.max(np.abs(want))
        assert results[True][0].tobytes() == results[False][0].tobytes() == results[False][1].tobytes()
        r.ctx.set_inputs_resident(True)
        s = torch.cuda.Stream()
        s.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(s):
            step()
        torch.cuda.current_stream().wait_stream(s)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            step()
        for _ in range(10):
            y.copy_(y_in)
            g.replay()
            torch.cuda.synchronize()
            assert y.cpu().numpy().tobytes() == results[True][0].tobytes()
        assert r.ctx.device_status() == 0
    finally:
        r.close()


def test_inputs_resident_hint_with_grouped_projections():
    # q, k and v of a layer in one launch, then o, several layers back to back, hint on: equal to the oracle
    # and to the run without the hint
    rng = np.random.default_rng(77)
    N, T, d = 48, 64, 512
    ranks = rng.choice([8, 16, 64], size=N)
    probs = [random_problem(950 + i, T=T, d_in=d, d_out=d, ranks=ranks) for i in range(8)]
    ids = probs[0]["ids"]
    ctx = P.Context(T, N)
    try:
        for i, p in enumerate(probs):
            ctx.register_pool(i // 4, i % 4, d, d, p["ranks"], p["scales"], p["A"], p["B"])
        x = bits_to_dev(probs[0]["x"])
        ids_t = torch.from_numpy(ids).to(DEV)
        outs = {}
        for hint in (False, True):
            ctx.set_inputs_resident(hint)
            ys = [torch.zeros((T, d), dtype=torch.float32, device=DEV) for _ in probs]
            ctx.bucket(ids_t, N)
            for layer in range(2):
                ctx.lora_delta_group([x, x, x], ids_t, [layer] * 3, [0, 1, 2], ys[4 * layer:4 * layer + 3])
                ctx.lora_delta(x, ids_t, layer, 3, ys[4 * layer + 3])
            torch.cuda.synchronize()
            outs[hint] = [y.cpu().numpy() for y in ys]
        for i, p in enumerate(probs):
            q = dict(p)
            q["ids"], q["x"] = ids, probs[0]["x"]
            ref = oracle.lora_delta(q["x"], q["ids"], q["ranks"], q["scales"], q["A"], q["B"], d, np.zeros((T, d), np.float32))
            assert rel_err(outs[True][i], ref) <= TOL_FP32_PATH
            assert outs[True][i].tobytes() == outs[False][i].tobytes()
        assert ctx.device_status() == 0
    finally:
        ctx.close()


def test_a_step_that_uses_both_kinds_of_mixed_rank_launch():
    # 400 tokens on a pool of mixed ranks: q, k and v grouped make 1200 rows (one launch per rank class, class lists
    # in bucket order), o alone 400 rows (one launch for all classes, lists ordered by token count).  Both sorts are
    # kept side by side: the first step sorts twice, later steps on the same bucket not at all; results are
    # bit-identical from step to step and equal to the oracle.
    rng = np.random.default_rng(911)
    N, T, d = 40, 400, 264
    ranks = rng.choice([8, 16, 32, 64, 128], size=N)
    probs = [random_problem(912 + j, T=T, d_in=d, d_out=d, ranks=ranks) for j in range(4)]
    ids_np = probs[0]["ids"].copy()
    ids_np[:160] = np.repeat(np.arange(40, dtype=np.int32), 4)        # units of four tokens next to single ones
    for pr in probs:
        pr["ids"], pr["x"] = ids_np, probs[0]["x"]
    ctx = P.Context(T, N)
    try:
        for j, pr in enumerate(probs):
            ctx.register_pool(0, j, d, d, pr["ranks"], pr["scales"], pr["A"], pr["B"])
        ctx.set_path(P.PATH_FUSED)
        ids = torch.from_numpy(ids_np).to(DEV)
        x = bits_to_dev(probs[0]["x"])
        ctx.bucket(ids, N)
        n_classes = len(set(int(r) for r in ranks))
        first = None
        for step in range(3):
            ys = [torch.from_numpy(probs[j]["y_in"]).to(DEV) for j in range(4)]
            n0 = ctx.launch_count()
            ctx.lora_delta_group([x, x, x], ids, [0, 0, 0], [0, 1, 2], ys[:3])
            ctx.lora_delta(x, ids, 0, 3, ys[3])
            torch.cuda.synchronize()
            sorts = 2 if step == 0 else 0
            assert ctx.launch_count() - n0 == sorts + n_classes + 1, step
            got = [y.cpu().numpy() for y in ys]
            if first is None:
                first = got
            for j in range(4):
                assert got[j].tobytes() == first[j].tobytes(), (step, j)
        for j in range(4):
            ref = _oracle(probs[j], y_in=probs[j]["y_in"])
            delta = np.max(np.abs(ref - probs[j]["y_in"]))
            assert np.max(np.abs(first[j] - ref)) <= TOL_FP32_PATH * delta + 1e-6 * np.max(np.abs(ref)), j
        assert ctx.device_status() == 0
    finally:
        ctx.close()

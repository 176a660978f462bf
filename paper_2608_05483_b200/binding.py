"""ctypes binding of the C ABI in include/plora.h.

Argument marshalling only: every step of the path runs in the CUDA library.
The module-level `plora_*` functions mirror the C entry points one to one
(pointers as ints, status codes returned); `Context` wraps them for torch
tensors and raises `PloraError` on a non-zero status.  There is no CPU
fallback: if the shared library is missing or cannot be loaded, import of the
functions fails loudly.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import numpy as np

from . import _build

OK = 0
ERR_INVALID_ARG = -1
ERR_NOT_REGISTERED = -2
ERR_BAD_ADAPTER_ID = -3
ERR_WORKSPACE = -4
ERR_CUDA = -5
ERR_TIMEOUT = -6
ERR_UNSUPPORTED = -7
ERR_DEBUG_CHECK = -8

PATH_AUTO, PATH_UNFUSED, PATH_FUSED, PATH_SGMV, PATH_SGMV_SPLIT = 0, 1, 2, 3, 4

EXPORTS = (
    "plora_create", "plora_destroy", "plora_pool_slab_bytes", "plora_register_pool", "plora_pool_max_rank",
    "plora_bucket", "plora_bucket_view", "plora_lora_delta", "plora_lora_delta_group", "plora_shrink", "plora_expand",
    "plora_shrink_m16", "plora_expand_m16", "plora_set_input_type",
    "plora_lora_delta_host", "plora_lora_delta_host_async", "plora_host_sync", "plora_lora_delta_noalloc", "plora_set_path", "plora_device_status", "plora_launch_count", "plora_status_string",
    "plora_cost_model", "plora_attn_workspace_bytes", "plora_attn_decode", "plora_attn_status", "plora_attn_set_debug",
    "plora_set_wait_limit", "plora_set_test_hook", "plora_set_inputs_resident", "plora_stream_read",
)

HOOK_NONE, HOOK_WITHHOLD_RELEASE, HOOK_MAX_CYCLES = 0, 1, 1 << 24


class PoolDesc(ctypes.Structure):
    _fields_ = [
        ("layer", ctypes.c_int32), ("proj", ctypes.c_int32),
        ("d_in", ctypes.c_int32), ("d_out", ctypes.c_int32),
        ("n_adapters", ctypes.c_int32), ("ab_on_device", ctypes.c_int32),
        ("ranks", ctypes.c_void_p), ("scales", ctypes.c_void_p),
        ("A", ctypes.c_void_p), ("B", ctypes.c_void_p),
    ]


class CostHw(ctypes.Structure):
    _fields_ = [(n, ctypes.c_double) for n in ("c_gpu", "w_gpu", "c_dev", "w_dram", "n_dev", "l_link", "w_link")]


class CostTerms(ctypes.Structure):
    _fields_ = [("t_gpu", ctypes.c_double * 4), ("t_dev_cpt", ctypes.c_double * 4), ("t_dev_trs", ctypes.c_double * 4),
                ("t_lora_gpu", ctypes.c_double), ("t_lora_dev", ctypes.c_double), ("t_lora", ctypes.c_double)]


class PloraError(RuntimeError):
    def __init__(self, status: int, where: str = ""):
        self.status = int(status)
        super().__init__(f"{where}: {status_string(status)} ({status})" if where else f"{status_string(status)} ({status})")


_lib = None


def _debug_build() -> bool:
    """PLORA_DEBUG_BUILD=1 in the environment selects the checked build of the library (same sources compiled with
    -DPLORA_DEBUG: kernels check every address against its buffer and report PLORA_ERR_DEBUG_CHECK)."""
    import os
    return os.environ.get("PLORA_DEBUG_BUILD", "") == "1"


def library_path() -> Path:
    return _build.LIB_DEBUG if _debug_build() else _build.LIB


def load(build_if_missing: bool = True):
    """Load libplora_b200.so (building it with nvcc first if it is not there)."""
    global _lib
    if _lib is not None:
        return _lib
    path = library_path()
    if not path.exists():
        if not build_if_missing:
            raise RuntimeError(f"{path} is missing: run __graft_entry__.build() (nvcc, sm_100a); there is no fallback path")
        _build.build(debug=_debug_build())
    lib = ctypes.CDLL(str(path))
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
    sig = {
        "plora_create": (i32, [ctypes.POINTER(vp), ctypes.c_int, i32, i32]),
        "plora_destroy": (i32, [vp]),
        "plora_pool_slab_bytes": (ctypes.c_size_t, [ctypes.POINTER(PoolDesc)]),
        "plora_register_pool": (i32, [vp, ctypes.POINTER(PoolDesc), vp, ctypes.c_size_t, vp]),
        "plora_pool_max_rank": (i32, [vp, i32, i32]),
        "plora_bucket": (i32, [vp, vp, i32, i32, vp]),
        "plora_bucket_view": (i32, [vp] + [ctypes.POINTER(vp)] * 5),
        "plora_lora_delta": (i32, [vp, vp, vp, i32, i32, i32, vp, vp]),
        "plora_lora_delta_group": (i32, [vp, i32, vp, vp, i32, vp, vp, vp, vp]),
        "plora_shrink": (i32, [vp, vp, vp, i32, i32, i32, vp, i32, vp]),
        "plora_expand": (i32, [vp, vp, i32, vp, i32, i32, i32, vp, vp]),
        "plora_shrink_m16": (i32, [vp, vp, vp, i32, i32, i32, vp, i32, vp]),
        "plora_expand_m16": (i32, [vp, vp, i32, vp, i32, i32, i32, vp, vp]),
        "plora_lora_delta_host": (i32, [vp, vp, vp, i32, i32, i32, vp, vp]),
        "plora_lora_delta_noalloc": (i32, [vp, vp, vp, i32, i32, i32, vp, vp]),
        "plora_lora_delta_host_async": (i32, [vp, i32, vp, vp, i32, vp, vp, vp, vp]),
        "plora_host_sync": (i32, [vp]),
        "plora_set_path": (i32, [vp, i32, i32]),
        "plora_set_input_type": (i32, [vp, i32]),
        "plora_device_status": (i32, [vp, vp, ctypes.POINTER(i32)]),
        "plora_launch_count": (i64, [vp]),
        "plora_status_string": (ctypes.c_char_p, [i32]),
        "plora_attn_workspace_bytes": (ctypes.c_size_t, [i32, i32, i32, i32]),
        "plora_attn_decode": (i32, [vp, vp, vp, vp, i32, i32, i32, i32, i32, ctypes.c_float, vp, vp, ctypes.c_size_t, vp]),
        "plora_attn_status": (i32, [vp, vp, ctypes.POINTER(i32)]),
        "plora_attn_set_debug": (i32, [vp, i64, i32, vp]),
        "plora_set_wait_limit": (i32, [vp, i64]),
        "plora_set_test_hook": (i32, [vp, i32]),
        "plora_set_inputs_resident": (i32, [vp, i32]),
        "plora_stream_read": (i32, [vp, ctypes.c_size_t, vp, ctypes.c_size_t, vp]),
        "plora_cost_model": (i32, [ctypes.POINTER(CostHw), i32, vp, vp, ctypes.c_double, ctypes.c_double, ctypes.c_double,
                                   ctypes.POINTER(CostTerms)]),
    }
    for name in EXPORTS:
        fn = getattr(lib, name)  # AttributeError here = the library does not export what the header declares
        fn.restype, fn.argtypes = sig[name]
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load().plora_status_string(int(status)).decode()


# ---- one-to-one wrappers (ints for pointers) ------------------------------------------
def plora_create(device: int, max_tokens: int, max_adapters: int):
    h = ctypes.c_void_p()
    rc = load().plora_create(ctypes.byref(h), int(device), int(max_tokens), int(max_adapters))
    return rc, h.value


def plora_destroy(ctx):
    return load().plora_destroy(ctx)


def plora_cost_model(hw: dict, ranks, batch, d: float, value_bytes: float, t_base: float):
    """(status, terms): the cost terms of the paper's four strategies (Section VI-B) as a dict of lists / floats.
    hw: c_gpu, w_gpu, c_dev, w_dram, n_dev, l_link, w_link.  batch: [n_adapters][4] request counts."""
    import numpy as np
    r = np.ascontiguousarray(ranks, np.int32)
    b = np.ascontiguousarray(batch, np.float64).reshape(len(r), 4)
    chw = CostHw(**{k: float(v) for k, v in hw.items()})
    out = CostTerms()
    rc = load().plora_cost_model(ctypes.byref(chw), len(r), r.ctypes.data, b.ctypes.data, float(d), float(value_bytes),
                                 float(t_base), ctypes.byref(out))
    terms = dict(t_gpu=list(out.t_gpu), t_dev_cpt=list(out.t_dev_cpt), t_dev_trs=list(out.t_dev_trs),
                 t_lora_gpu=out.t_lora_gpu, t_lora_dev=out.t_lora_dev, t_lora=out.t_lora)
    return rc, terms


def plora_attn_workspace_bytes(n_req: int, max_kv_len: int, n_kv_heads: int, q_per_kv: int) -> int:
    return int(load().plora_attn_workspace_bytes(n_req, max_kv_len, n_kv_heads, q_per_kv))


def plora_attn_decode(q_ptr, k_ptr, v_ptr, kv_len_ptr, n_req, max_kv_len, n_kv_heads, q_per_kv, head_dim, scale, out_ptr,
                      ws_ptr, ws_bytes, stream=0):
    return load().plora_attn_decode(q_ptr, k_ptr, v_ptr, kv_len_ptr, n_req, max_kv_len, n_kv_heads, q_per_kv, head_dim,
                                    float(scale), out_ptr, ws_ptr, ws_bytes, stream)


def plora_attn_status(ws_ptr, stream=0):
    v = ctypes.c_int32(0)
    rc = load().plora_attn_status(ws_ptr, stream, ctypes.byref(v))
    return rc, int(v.value)


def plora_attn_set_debug(ws_ptr, cycles: int, hook: int, stream=0):
    return load().plora_attn_set_debug(ws_ptr, int(cycles), int(hook), stream)


def plora_set_wait_limit(ctx, cycles: int):
    return load().plora_set_wait_limit(ctx, int(cycles))


def plora_set_test_hook(ctx, hook: int):
    return load().plora_set_test_hook(ctx, int(hook))


def plora_set_inputs_resident(ctx, resident: bool):
    return load().plora_set_inputs_resident(ctx, 1 if resident else 0)


def plora_stream_read(buf_ptr, nbytes: int, sink_ptr, sink_bytes: int, stream=0):
    return load().plora_stream_read(buf_ptr, int(nbytes), sink_ptr, int(sink_bytes), stream)


def attn_decode(q, k_cache, v_cache, kv_len, scale, out=None, workspace=None, stream=None):
    """Torch convenience: q bf16 [B, Hq, 128], k_cache / v_cache bf16 [B, Hkv, Lmax, 128], kv_len int32 [B] (all CUDA);
    returns (out fp32 [B, Hq, 128], workspace).  Pass the returned workspace back in to reuse it."""
    import torch
    B, Hq, d = q.shape
    Hkv, Lmax = int(k_cache.shape[1]), int(k_cache.shape[2])
    need = plora_attn_workspace_bytes(B, Lmax, Hkv, Hq // Hkv)
    if workspace is None:
        workspace = torch.zeros(need, dtype=torch.uint8, device=q.device)
    if out is None:
        out = torch.empty((B, Hq, d), dtype=torch.float32, device=q.device)
    _check(plora_attn_decode(q.data_ptr(), k_cache.data_ptr(), v_cache.data_ptr(), kv_len.data_ptr(), B, Lmax, Hkv, Hq // Hkv,
                             d, scale, out.data_ptr(), workspace.data_ptr(), int(workspace.numel()), _stream_handle(stream)),
           "plora_attn_decode")
    return out, workspace


def plora_pool_slab_bytes(desc: PoolDesc) -> int:
    return int(load().plora_pool_slab_bytes(ctypes.byref(desc)))


def plora_register_pool(ctx, desc: PoolDesc, slab_ptr: int, slab_bytes: int, stream: int = 0):
    return load().plora_register_pool(ctx, ctypes.byref(desc), slab_ptr, slab_bytes, stream)


def plora_pool_max_rank(ctx, layer: int, proj: int) -> int:
    return load().plora_pool_max_rank(ctx, layer, proj)


def plora_bucket(ctx, ids_ptr: int, n_tok: int, n_adapters: int, stream: int = 0):
    return load().plora_bucket(ctx, ids_ptr, n_tok, n_adapters, stream)


def plora_bucket_view(ctx):
    ptrs = [ctypes.c_void_p() for _ in range(5)]
    rc = load().plora_bucket_view(ctx, *[ctypes.byref(p) for p in ptrs])
    return rc, tuple(p.value for p in ptrs)


def plora_lora_delta(ctx, x_ptr: int, ids_ptr: int, n_tok: int, layer: int, proj: int, y_ptr: int, stream: int = 0):
    return load().plora_lora_delta(ctx, x_ptr, ids_ptr, n_tok, layer, proj, y_ptr, stream)


def plora_lora_delta_group(ctx, x_ptrs, ids_ptr, n_tok, layers, projs, y_ptrs, stream=0):
    """x_ptrs / y_ptrs: sequences of device pointers; layers / projs: sequences of ints (all of length n)."""
    n = len(x_ptrs)
    xs = (ctypes.c_void_p * n)(*x_ptrs)
    ys = (ctypes.c_void_p * n)(*y_ptrs)
    ls = (ctypes.c_int32 * n)(*layers)
    ps = (ctypes.c_int32 * n)(*projs)
    return load().plora_lora_delta_group(ctx, n, ctypes.cast(xs, ctypes.c_void_p), ids_ptr, n_tok,
                                         ctypes.cast(ls, ctypes.c_void_p), ctypes.cast(ps, ctypes.c_void_p),
                                         ctypes.cast(ys, ctypes.c_void_p), stream)


def plora_shrink(ctx, x_ptr, ids_ptr, n_tok, layer, proj, m_ptr, ldm, stream=0):
    return load().plora_shrink(ctx, x_ptr, ids_ptr, n_tok, layer, proj, m_ptr, ldm, stream)


def plora_expand(ctx, m_ptr, ldm, ids_ptr, n_tok, layer, proj, y_ptr, stream=0):
    return load().plora_expand(ctx, m_ptr, ldm, ids_ptr, n_tok, layer, proj, y_ptr, stream)


def plora_shrink_m16(ctx, x_ptr, ids_ptr, n_tok, layer, proj, m_ptr, ldm, stream=0):
    return load().plora_shrink_m16(ctx, x_ptr, ids_ptr, n_tok, layer, proj, m_ptr, ldm, stream)


def plora_expand_m16(ctx, m_ptr, ldm, ids_ptr, n_tok, layer, proj, y_ptr, stream=0):
    return load().plora_expand_m16(ctx, m_ptr, ldm, ids_ptr, n_tok, layer, proj, y_ptr, stream)


def plora_lora_delta_host(ctx, x_host_ptr, ids_host_ptr, n_tok, layer, proj, y_host_ptr, stream=0):
    return load().plora_lora_delta_host(ctx, x_host_ptr, ids_host_ptr, n_tok, layer, proj, y_host_ptr, stream)


def plora_lora_delta_host_async(ctx, x_host_ptr, ids_host_ptr, n_tok, layers, projs, y_host_ptrs, stream=0):
    n = len(layers)
    la = (ctypes.c_int32 * n)(*layers)
    pa = (ctypes.c_int32 * n)(*projs)
    ya = (ctypes.c_void_p * n)(*y_host_ptrs)
    return load().plora_lora_delta_host_async(ctx, n, x_host_ptr, ids_host_ptr, n_tok, la, pa, ya, stream)


def plora_host_sync(ctx):
    return load().plora_host_sync(ctx)


def plora_lora_delta_noalloc(ctx, x_ptr, ids_ptr, n_tok, layer, proj, y_ptr, stream=0):
    return load().plora_lora_delta_noalloc(ctx, x_ptr, ids_ptr, n_tok, layer, proj, y_ptr, stream)


def plora_set_path(ctx, path: int, sgmv_min_rows: int = 0):
    return load().plora_set_path(ctx, path, sgmv_min_rows)


def plora_device_status(ctx, stream: int = 0):
    v = ctypes.c_int32(0)
    rc = load().plora_device_status(ctx, stream, ctypes.byref(v))
    return rc, int(v.value)


def plora_launch_count(ctx) -> int:
    return int(load().plora_launch_count(ctx))


# ---- torch-facing convenience layer -------------------------------------------------------
class _DevArray:
    """Exposes a raw device pointer to torch through the CUDA array interface."""

    def __init__(self, ptr: int, n: int, typestr: str = "<i4"):
        self.__cuda_array_interface__ = {"shape": (n,), "typestr": typestr, "data": (ptr, False), "version": 2}


def _stream_handle(stream) -> int:
    import torch
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def _check(rc: int, where: str):
    if rc != OK:
        raise PloraError(rc, where)


def _data_ptr(t) -> int:
    if isinstance(t, np.ndarray):
        return int(t.ctypes.data)
    return int(t.data_ptr())


class Context:
    """One library context (one device, one stream at a time)."""

    def __init__(self, max_tokens: int, max_adapters: int, device: int = 0):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("no CUDA device: this library has no CPU path")
        rc, h = plora_create(device, max_tokens, max_adapters)
        _check(rc, "plora_create")
        self._h = h
        self.device = device
        self.max_tokens, self.max_adapters = max_tokens, max_adapters
        self._slabs = {}
        self._n_tok = 0
        self._n_adapters = 0

    def close(self):
        if getattr(self, "_h", None):
            plora_destroy(self._h)
            self._h = None
            self._slabs.clear()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def handle(self):
        return self._h

    def register_pool(self, layer, proj, d_in, d_out, ranks, scales, A, B, stream=None):
        """A, B: per-adapter lists of bf16 matrices [d_in, r_a] / [r_a, d_out]: torch tensors
        (all on the device, or all on the host) or numpy uint16 bit patterns.  Returns the slab tensor."""
        import torch
        n = len(A)
        ranks = np.ascontiguousarray(ranks, dtype=np.int32)
        scales = np.ascontiguousarray(scales, dtype=np.float32)
        assert len(B) == n and ranks.shape == (n,) and scales.shape == (n,)
        on_dev = bool(n) and (not isinstance(A[0], np.ndarray)) and A[0].is_cuda
        keep = []
        pa = (ctypes.c_void_p * n)()
        pb = (ctypes.c_void_p * n)()
        for a in range(n):
            ma, mb = A[a], B[a]
            if isinstance(ma, np.ndarray):
                ma = np.ascontiguousarray(ma, dtype=np.uint16)
                mb = np.ascontiguousarray(mb, dtype=np.uint16)
            else:
                assert ma.is_cuda == on_dev and mb.is_cuda == on_dev and ma.dtype in (torch.bfloat16, torch.float16)
                ma, mb = ma.contiguous(), mb.contiguous()
            assert tuple(ma.shape) == (d_in, int(ranks[a])), (a, tuple(ma.shape))
            assert tuple(mb.shape) == (int(ranks[a]), d_out), (a, tuple(mb.shape))
            keep += [ma, mb]
            pa[a], pb[a] = _data_ptr(ma), _data_ptr(mb)
        desc = PoolDesc(layer, proj, d_in, d_out, n, 1 if on_dev else 0, ranks.ctypes.data, scales.ctypes.data,
                        ctypes.cast(pa, ctypes.c_void_p).value, ctypes.cast(pb, ctypes.c_void_p).value)
        nbytes = plora_pool_slab_bytes(desc)
        if nbytes == 0:
            raise PloraError(ERR_UNSUPPORTED, "plora_pool_slab_bytes")
        slab = torch.empty(nbytes, dtype=torch.uint8, device=f"cuda:{self.device}")
        assert slab.data_ptr() % 256 == 0
        _check(plora_register_pool(self._h, desc, slab.data_ptr(), nbytes, _stream_handle(stream)), "plora_register_pool")
        del keep
        self._slabs[(layer, proj)] = slab
        return slab

    def pool_max_rank(self, layer, proj) -> int:
        r = plora_pool_max_rank(self._h, layer, proj)
        if r < 0:
            raise PloraError(r, "plora_pool_max_rank")
        return r

    def bucket(self, ids, n_adapters: int, stream=None):
        self._n_tok, self._n_adapters = int(ids.numel()), int(n_adapters)
        _check(plora_bucket(self._h, ids.data_ptr(), self._n_tok, n_adapters, _stream_handle(stream)), "plora_bucket")

    def bucket_view(self):
        """Host copies of the current bucket: dict(perm, seg_adapter, seg_start, n_seg, n_active)."""
        import torch
        rc, (perm, seg_adapter, seg_start, n_seg, n_active) = plora_bucket_view(self._h)
        _check(rc, "plora_bucket_view")
        torch.cuda.synchronize()
        cap = min(self._n_tok, self._n_adapters)
        dev = f"cuda:{self.device}"

        def grab(ptr, n):
            if n == 0:
                return np.zeros(0, np.int32)
            return torch.as_tensor(_DevArray(ptr, n), device=dev).cpu().numpy().copy()

        return dict(perm=grab(perm, self._n_tok), seg_adapter=grab(seg_adapter, cap), seg_start=grab(seg_start, cap + 1),
                    n_seg=int(grab(n_seg, 1)[0]), n_active=int(grab(n_active, 1)[0]))

    def lora_delta(self, x, ids, layer, proj, y, stream=None):
        _check(plora_lora_delta(self._h, x.data_ptr(), ids.data_ptr(), int(ids.numel()), layer, proj, y.data_ptr(),
                                _stream_handle(stream)), "plora_lora_delta")

    def lora_delta_group(self, xs, ids, layers, projs, ys, stream=None):
        """Independent projections (q/k/v of a layer, up/gate) in one call; same-shape pools share a launch."""
        _check(plora_lora_delta_group(self._h, [t.data_ptr() for t in xs], ids.data_ptr(), int(ids.numel()),
                                      list(layers), list(projs), [t.data_ptr() for t in ys], _stream_handle(stream)),
               "plora_lora_delta_group")

    def shrink(self, x, ids, layer, proj, m, stream=None):
        _check(plora_shrink(self._h, x.data_ptr(), ids.data_ptr(), int(ids.numel()), layer, proj, m.data_ptr(),
                            int(m.shape[1]), _stream_handle(stream)), "plora_shrink")

    def expand(self, m, ids, layer, proj, y, stream=None):
        _check(plora_expand(self._h, m.data_ptr(), int(m.shape[1]), ids.data_ptr(), int(ids.numel()), layer, proj,
                            y.data_ptr(), _stream_handle(stream)), "plora_expand")

    def shrink_m16(self, x, ids, layer, proj, m_bf16, stream=None):
        _check(plora_shrink_m16(self._h, x.data_ptr(), ids.data_ptr(), int(ids.numel()), layer, proj, m_bf16.data_ptr(),
                                int(m_bf16.shape[1]), _stream_handle(stream)), "plora_shrink_m16")

    def expand_m16(self, m_bf16, ids, layer, proj, y, stream=None):
        _check(plora_expand_m16(self._h, m_bf16.data_ptr(), int(m_bf16.shape[1]), ids.data_ptr(), int(ids.numel()), layer,
                                proj, y.data_ptr(), _stream_handle(stream)), "plora_expand_m16")

    def lora_delta_host(self, x_host, ids_host, layer, proj, y_host, stream=None):
        """x_host / ids_host / y_host: CPU torch tensors (pinned or not) or numpy arrays; y_host is updated in place."""
        n_tok = int(ids_host.shape[0])
        _check(plora_lora_delta_host(self._h, _data_ptr(x_host), _data_ptr(ids_host), n_tok, layer, proj,
                                     _data_ptr(y_host), _stream_handle(stream)), "plora_lora_delta_host")

    def lora_delta_host_async(self, x_host, ids_host, layers, projs, ys_host, stream=None):
        """Queues y_host[g] += delta of pool (layers[g], projs[g]) for projections that share x_host;
        the results are in host memory after host_sync().  The host tensors must stay alive and
        untouched until then."""
        n_tok = int(ids_host.shape[0])
        _check(plora_lora_delta_host_async(self._h, _data_ptr(x_host), _data_ptr(ids_host), n_tok, list(layers), list(projs),
                                           [_data_ptr(y) for y in ys_host], _stream_handle(stream)),
               "plora_lora_delta_host_async")

    def host_sync(self):
        _check(plora_host_sync(self._h), "plora_host_sync")

    def lora_delta_noalloc(self, x, ids, layer, proj, y, stream=None):
        """The delta for callers that must not allocate: same result as lora_delta, with the
        intermediate m in the library's fixed scratch array (see plora_lora_delta_noalloc)."""
        _check(plora_lora_delta_noalloc(self._h, x.data_ptr(), ids.data_ptr(), int(ids.numel()), layer, proj,
                                        y.data_ptr(), _stream_handle(stream)), "plora_lora_delta_noalloc")

    def set_path(self, path: int, sgmv_min_rows: int = 0):
        _check(plora_set_path(self._h, path, sgmv_min_rows), "plora_set_path")

    def set_wait_limit(self, cycles: int):
        _check(plora_set_wait_limit(self._h, cycles), "plora_set_wait_limit")

    def set_test_hook(self, hook: int):
        _check(plora_set_test_hook(self._h, hook), "plora_set_test_hook")

    def set_inputs_resident(self, resident: bool):
        _check(plora_set_inputs_resident(self._h, resident), "plora_set_inputs_resident")

    def set_input_type(self, fp16: bool):
        _check(load().plora_set_input_type(self._h, 1 if fp16 else 0), "plora_set_input_type")

    def device_status(self, stream=None) -> int:
        rc, v = plora_device_status(self._h, _stream_handle(stream))
        _check(rc, "plora_device_status")
        return v

    def launch_count(self) -> int:
        return plora_launch_count(self._h)

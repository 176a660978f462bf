"""The C-ABI library builds, loads without a GPU and exports every symbol the header declares."""
import ctypes
import re
from pathlib import Path

import paper_2608_05483_b200 as P

ROOT = Path(__file__).resolve().parent.parent


def _declared():
    text = (ROOT / "include" / "plora.h").read_text()
    return sorted(set(re.findall(r"PLORA_API[^;(]*?\b(plora_\w+)\s*\(", text)))


def test_header_declares_the_named_calls():
    names = _declared()
    for must in ("plora_register_pool", "plora_bucket", "plora_lora_delta", "plora_shrink", "plora_expand",
                 "plora_create", "plora_destroy", "plora_lora_delta_host"):
        assert must in names


def test_library_exports_every_declared_symbol():
    lib = P.load()
    raw = ctypes.CDLL(str(P.library_path()))
    for name in _declared():
        assert hasattr(raw, name), name
    assert sorted(P.EXPORTS) == _declared()
    assert lib is P.load()


def test_status_strings_and_host_side_argument_checks():
    assert P.status_string(P.OK) == "ok"
    assert "adapter" in P.status_string(P.ERR_BAD_ADAPTER_ID)
    # no compute without a GPU: these return before touching the device
    rc, h = P.plora_create(0, 0, 16)
    assert rc == P.ERR_INVALID_ARG and h is None
    rc, h = P.plora_create(0, 16, 10 ** 9)
    assert rc == P.ERR_UNSUPPORTED
    assert P.plora_destroy(None) == P.ERR_INVALID_ARG
    assert P.plora_launch_count(None) == -1


def test_slab_size_matches_layout_rules():
    import numpy as np
    ranks = np.array([16, 8, 64, 3], np.int32)
    d = P.PoolDesc(0, 0, 4096, 4096, 4, 0, ranks.ctypes.data, None, None, None)
    # per adapter: tiles of 16 KiB (8 KiB when the padded rank is 8) covering d_in and d_out
    want = (8 + 8) * 16384 + (8 + 8) * 8192 + (32 + 32) * 16384 + (8 + 8) * 8192
    assert P.plora_pool_slab_bytes(d) == want
    bad = P.PoolDesc(0, 0, 4100, 4096, 4, 0, ranks.ctypes.data, None, None, None)
    assert P.plora_pool_slab_bytes(bad) == 0
    ranks[0] = 129
    assert P.plora_pool_slab_bytes(d) == 0

"""The C-ABI library builds, loads and exports every symbol the header declares (no GPU)."""
import ctypes
import os
import re

import pytest

from paper_2506_07533_b200 import binding as mq
from paper_2506_07533_b200 import build as mqbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    mqbuild.build()
    return mq.lib()


def declared_functions():
    src = open(os.path.join(ROOT, "include", "moqae.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(moqae_[a-z_0-9]+)\s*\(", src)))


def test_exports_match_header(lib):
    names = declared_functions()
    assert len(names) >= 11
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(mq.EXPORTS) == [n for n in names if n in mq.EXPORTS]
    assert set(names) == set(mq.EXPORTS)


def test_version_and_error_strings(lib):
    assert lib.moqae_version() >= 100
    assert lib.moqae_error_string(0) == b"ok"
    for code in range(-7, 0):
        assert len(lib.moqae_error_string(code)) > 3


def test_struct_sizes_match_header():
    assert ctypes.sizeof(mq.MoqaeConfig) == 19 * 4
    assert ctypes.sizeof(mq.MoqaeCache) == 4 * 8 + 4 * 8 + 8 * 8


def test_cache_bytes_closed_form(lib):
    cfg = mq.make_config(n_layers=2, n_q_heads=8, n_kv_heads=4, chunk=128, dtype=1, d_in=1024,
                         max_tokens=4096, batch=3, rs_group=2)
    sizes = mq.moqae_cache_bytes(cfg, [5, 6, 7, 8])
    per = 2 * 3 * 4
    assert sizes[:4] == [per * 5 * 128 * 96, per * 6 * 128 * 160, per * 7 * 128 * 288, per * 8 * 128 * 512]
    assert sizes[4] == 1 * 3 * 32 and sizes[5] == 4 * sizes[4] and sizes[7] == 16 * sizes[4]
    assert sizes[6] == 3 * 16 and sizes[8] == sizes[9] == per * 128 * 256 and sizes[10] == 2 * 3 * 4


def test_host_side_argument_errors(lib):
    bad = mq.make_config(n_layers=1, n_q_heads=8, n_kv_heads=8, chunk=100, dtype=0, d_in=1024,
                         max_tokens=4096, batch=1)
    with pytest.raises(mq.MoqaeError) as e:
        mq.moqae_cache_bytes(bad, [1, 1, 1, 1])
    assert e.value.code == mq.ERR_UNSUPPORTED          # chunk not a multiple of 32
    bad = mq.make_config(n_layers=1, n_q_heads=8, n_kv_heads=3, chunk=128, dtype=0, d_in=1024,
                         max_tokens=4096, batch=1)
    with pytest.raises(mq.MoqaeError) as e:
        mq.moqae_cache_bytes(bad, [1, 1, 1, 1])
    assert e.value.code == mq.ERR_INVALID_ARG
    ok = mq.make_config(n_layers=1, n_q_heads=8, n_kv_heads=8, chunk=128, dtype=0, d_in=1024,
                        max_tokens=4096, batch=1)
    with pytest.raises(mq.MoqaeError) as e:
        mq.moqae_cache_bytes(ok, [1, -1, 1, 1])
    assert e.value.code == mq.ERR_INVALID_ARG
    # null cache / misaligned pointers are rejected before any launch
    cache = mq.MoqaeCache()
    rc = lib.moqae_decode_attn(ctypes.byref(ok), ctypes.c_void_p(16), 0, ctypes.byref(cache),
                               ctypes.c_void_p(16), ctypes.c_float(0), ctypes.c_void_p(16), 0, None)
    assert rc == mq.ERR_INVALID_ARG
    bufs = (ctypes.c_void_p * 12)(*[4096 + 16 * i for i in range(12)])
    bufs[2] = 4097
    cap = (ctypes.c_int64 * 4)(1, 1, 1, 1)
    assert lib.moqae_cache_bind(ctypes.byref(ok), cap, bufs, ctypes.byref(cache)) == mq.ERR_MISALIGNED


def test_table_validator_on_host_arrays(lib):
    """The index-table checker (host arithmetic, no GPU): tables made by the oracle's slot rule pass;
    a wrong slot, a slot beyond its pool, an unknown width and a wrong count are each reported at
    their position."""
    import numpy as np
    from oracle import moqae_oracle as O
    rs = np.random.RandomState(0)
    bmap = rs.randint(0, 4, size=(3, 40)).astype(np.uint8)
    slot, count = O.assign_slots(bmap)
    cap = [int(count[:, w].max()) for w in range(4)]
    assert mq.moqae_validate_tables_host(bmap, slot, count, 40, cap)[0] == mq.OK
    assert mq.moqae_validate_tables_host(bmap, slot, np.zeros_like(count), 0, cap)[0] == mq.OK      # an empty context
    bad = slot.copy(); bad[1, 17] += 1
    assert mq.moqae_validate_tables_host(bmap, bad, count, 40, cap) == (mq.ERR_CORRUPT_TABLE, 1, 17)
    assert mq.moqae_validate_tables_host(bmap, bad, count, 17, cap)[0] == mq.ERR_CORRUPT_TABLE     # count row no longer fits
    small = list(cap); small[int(bmap[2, 39])] = int(slot[2, 39])                                  # last chunk's slot == capacity
    rc, r, c = mq.moqae_validate_tables_host(bmap, slot, count, 40, small)
    assert rc == mq.ERR_CORRUPT_TABLE and c >= 0
    m2 = bmap.copy(); m2[0, 3] = 7
    assert mq.moqae_validate_tables_host(m2, slot, count, 40, cap) == (mq.ERR_CORRUPT_TABLE, 0, 3)
    k2 = count.copy(); k2[2, 1] += 1
    assert mq.moqae_validate_tables_host(bmap, slot, k2, 40, cap) == (mq.ERR_CORRUPT_TABLE, 2, -1)

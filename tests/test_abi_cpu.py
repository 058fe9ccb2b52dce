"""CPU-only checks of the C ABI: the library loads, exports what the header declares,
and its host-side logic (strategy validation, slot numbering, byte accounting, state
errors) is exact.  No kernel is launched and no CUDA device is needed."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
from paper_2410_18517_b200 import binding as kb
from paper_2410_18517_b200 import build as kbuild
from synth_inputs import random_share_map

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    kbuild.build()


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "kvs.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(kvs_[a-z_]+)\s*\(", header))
    assert declared == set(kb.EXPORTS)
    lib = ctypes.CDLL(kb.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), name


def test_status_strings():
    assert kb.kvs_status_string(kb.KVS_OK) == "ok"
    assert len({kb.kvs_status_string(s) for s in range(8)}) == 8


def _create(L=4, Hq=4, Hkv=4, D=64, B=2, S=136, dt=kb.KVS_F32, scale=0.0):
    return kb.kvs_create(L, Hq, Hkv, D, B, S, dt, scale, 0)


@pytest.mark.parametrize("kw", [dict(L=0), dict(Hq=3, Hkv=2), dict(Hq=12, Hkv=4), dict(D=96), dict(B=0), dict(S=0),
                                dict(dt=2), dict(scale=-1.0), dict(Hq=16, Hkv=1)])
def test_create_rejects_bad_configs(kw):
    with pytest.raises(kb.KvsError) as e:
        _create(**kw)
    assert e.value.status == kb.KVS_ERR_INVALID_ARG


def test_group_sizes():
    for G in range(1, 9):
        c = _create(Hq=2 * G, Hkv=2, D=128, dt=kb.KVS_BF16)      # every group size up to 8 with bf16
        kb.kvs_destroy(c)
    for G in (1, 2, 4, 8):
        kb.kvs_destroy(_create(Hq=2 * G, Hkv=2, dt=kb.KVS_F32))
    for G in (3, 5, 6, 7):
        with pytest.raises(kb.KvsError):
            _create(Hq=2 * G, Hkv=2, dt=kb.KVS_F32)


def test_identity_map_by_default_and_tiny_strategy():
    c = _create()
    assert kb.kvs_num_slots(c) == 4
    assert [kb.kvs_slot_of_layer(c, l) for l in range(4)] == [0, 1, 2, 3]
    kb.kvs_set_share_map(c, [0, 1, 2, 1])
    assert kb.kvs_num_slots(c) == 3
    assert [kb.kvs_slot_of_layer(c, l) for l in range(4)] == [0, 1, 2, 1]
    kb.kvs_destroy(c)


def test_share_map_validation():
    c = _create()
    for bad in ([0, 2, 2, 3], [1, 1, 2, 3], [0, -1, 2, 3], [0, 1, 2, 4]):
        with pytest.raises(kb.KvsError) as e:
            kb.kvs_set_share_map(c, bad)
        assert e.value.status == kb.KVS_ERR_BAD_SHARE_MAP
    assert kb.kvs_num_slots(c) == 4          # a rejected map changes nothing
    kb.kvs_destroy(c)


def test_slot_table_matches_oracle_on_random_strategies_with_chains():
    rng = np.random.default_rng(1)
    for _ in range(100):
        L = int(rng.integers(1, 40))
        sm = [int(rng.integers(0, l + 1)) for l in range(L)]
        c = _create(L=L)
        kb.kvs_set_share_map(c, sm)
        n, root, slot = oracle.slot_table(sm)
        assert kb.kvs_num_slots(c) == n
        assert [kb.kvs_slot_of_layer(c, l) for l in range(L)] == slot.tolist()
        kb.kvs_destroy(c)


@pytest.mark.parametrize("L,P", [(32, 4), (32, 8), (32, 12), (40, 5), (40, 10), (40, 15), (48, 6), (48, 12), (48, 18),
                                 (80, 10), (80, 20)])
def test_slot_count_is_layers_minus_shared(L, P):
    c = _create(L=L)
    kb.kvs_set_share_map(c, random_share_map(L, P, 0))
    assert kb.kvs_num_slots(c) == L - P
    kb.kvs_destroy(c)


def test_pool_bytes_and_plane_offsets():
    # 7B-shaped: one slot = 2 planes of 8*32*4096*128 bf16 = 256 MiB each
    c = kb.kvs_create(32, 32, 32, 128, 8, 4096, kb.KVS_BF16, 0.0, 0)
    pool, ws = kb.kvs_required_bytes(c)
    assert pool == 32 * 2 * 256 * 2**20
    kb.kvs_set_share_map(c, random_share_map(32, 8, 2))
    pool2, _ = kb.kvs_required_bytes(c)
    assert pool2 == 24 * 2 * 256 * 2**20 and pool2 * 32 == pool * 24
    assert kb.kvs_row_stride(c) == 4096
    assert kb.kvs_plane_offset(c, 0, 0) == 0
    assert kb.kvs_plane_offset(c, 0, 1) == 256 * 2**20
    assert kb.kvs_plane_offset(c, 23, 1) == 47 * 256 * 2**20
    with pytest.raises(kb.KvsError):
        kb.kvs_plane_offset(c, 24, 0)
    assert ws < 64 * 2**20
    kb.kvs_destroy(c)
    # capacity is rounded up to 128 rows: the tiny case asks for 136 and gets 256
    c = _create()
    assert kb.kvs_row_stride(c) == 256
    pool, _ = kb.kvs_required_bytes(c)
    assert pool == 4 * 2 * (2 * 4 * 256 * 64 * 4)
    kb.kvs_destroy(c)


def test_calls_before_bind_report_state():
    c = _create()
    for fn in (lambda: kb.kvs_append(c, 0, 16, 16, 2, 1),
               lambda: kb.kvs_decode_attention(c, 0, 16, 16, 2),
               lambda: kb.kvs_last_device_status(c)):
        with pytest.raises(kb.KvsError) as e:
            fn()
        assert e.value.status == kb.KVS_ERR_STATE
    assert kb.kvs_seq_len(c, 3) == 0
    kb.kvs_reset(c)
    kb.kvs_destroy(c)


def test_bind_rejects_small_or_misaligned_buffers_without_touching_cuda():
    c = _create()
    pool, ws = kb.kvs_required_bytes(c)
    with pytest.raises(kb.KvsError) as e:
        kb.kvs_bind_memory(c, 4096, pool - 1, 8192, ws)
    assert e.value.status == kb.KVS_ERR_OOM
    with pytest.raises(kb.KvsError) as e:
        kb.kvs_bind_memory(c, 4096 + 8, pool, 8192, ws)
    assert e.value.status == kb.KVS_ERR_INVALID_ARG
    kb.kvs_destroy(c)


def test_options_and_null_arguments():
    c = _create()
    kb.kvs_set_option(c, kb.KVS_OPT_MAX_CTAS, 7)
    with pytest.raises(kb.KvsError):
        kb.kvs_set_option(c, kb.KVS_OPT_MAX_CTAS, 100000)
    with pytest.raises(kb.KvsError):
        kb.kvs_set_option(c, 99, 0)
    kb.kvs_set_option(c, kb.KVS_OPT_HOST_CHUNKS, 3)
    for bad in (0, 9):
        with pytest.raises(kb.KvsError):
            kb.kvs_set_option(c, kb.KVS_OPT_HOST_CHUNKS, bad)
    with pytest.raises(kb.KvsError):
        kb.kvs_slot_of_layer(c, 4)
    lib = kb.load()
    assert lib.kvs_destroy(None) == kb.KVS_ERR_INVALID_ARG
    assert lib.kvs_create(None, None) == kb.KVS_ERR_INVALID_ARG
    assert lib.kvs_read_roof(None, 32768, None, 0, None) == kb.KVS_ERR_INVALID_ARG
    kb.kvs_destroy(c)

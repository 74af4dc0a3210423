"""Host-side checks of the C ABI that need no GPU: the library builds, loads, exports every symbol
the header declares, and its layout arithmetic agrees with the oracle's independent restatement."""
import ctypes as C
import itertools
import os
import re

import pytest

from oracle import loco_oracle as orc
from paper_2407_04480_b200 import build as loco_build
from paper_2407_04480_b200 import loco

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    loco_build.build()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "loco.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(loco_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_functions()
    assert "loco_compensate_quantize_pack" in names and "loco_unpack_dequant_reduce" in names
    assert "loco_state_init" in names and "loco_state_reset" in names
    L = C.CDLL(loco.LIB_PATH)
    for name in names:
        assert hasattr(L, name), "symbol %s declared in loco.h but not exported" % name
    assert sorted(loco.EXPORTS) == names


def test_binding_has_the_same_names():
    for name in declared_functions():
        if name in ("loco_status_string",):
            continue
        assert hasattr(loco, name), name


def test_sizes_agree_with_the_oracle_layout():
    ns = [0, 1, 255, 256, 257, 1000, 4096, 65537, 25_000_000, 13_015_864_320]
    for bits, mode, B, P, fmt in itertools.product((1, 2, 4, 8), (0, 1), (32, 256, 4096), (1, 3, 8, 64), (0, 1, 2, 3)):
        if mode == 1 and fmt == 3:
            continue
        kw = dict(bits=bits, scale_mode=mode, block_size=B, s=2.0 ** 14, s_e=2.0 ** 16, beta=0.5, reset_period=512,
                  state_fmt=fmt, grad_dtype=1, out_dtype=1, num_partitions=P)
        g, o = loco.Config(**kw), orc.OracleConfig(**kw)
        for n in ns:
            assert loco.loco_state_bytes(g, n) == orc.state_bytes(o, n)
            assert loco.loco_packed_bytes(g, n) == orc.packed_bytes(o, n)
            assert loco.loco_partition_bytes(g, n) == orc.partition_bytes(o, n)
            assert loco.loco_partition_capacity(g, n) == orc.partition_capacity(o, n)
            for j in (0, P // 2, P - 1):
                assert loco.loco_partition_elems(g, n, j) == orc.partition_elems(o, n, j)
            assert loco.loco_partition_bytes(g, n) % 128 == 0


def test_bad_configurations_are_rejected():
    good = dict(bits=4, s=2.0 ** 14, s_e=2.0 ** 16, beta=0.5)
    assert loco.loco_config_check(loco.Config(**good)) == loco.OK
    for bad in (dict(bits=3), dict(bits=16), dict(s=0.0), dict(s=float("inf")), dict(s_e=-1.0), dict(beta=1.5),
                dict(beta=float("nan")), dict(reset_period=-1), dict(num_partitions=0), dict(state_fmt=7),
                dict(grad_dtype=2), dict(scale_mode=1, block_size=48), dict(scale_mode=1, block_size=16),
                dict(scale_mode=1, state_fmt=3), dict(scale_mode=1, block_size=8192), dict(bits=1, rounding=1),
                dict(bits=0)):
        cfg = loco.Config(**{**good, **bad})
        assert loco.loco_config_check(cfg) == loco.ERR_ARG, bad
        assert loco.loco_state_bytes(cfg, 1000) == 0 and loco.loco_packed_bytes(cfg, 1000) == 0
    # every block size the layout defines is one the kernels run: powers of two from 32 to 4096; and every code width
    for B in (32, 64, 128, 256, 512, 1024, 2048, 4096):
        for bits in (1, 2, 4, 8):
            assert loco.loco_config_check(loco.Config(bits=bits, scale_mode=1, block_size=B)) == loco.OK
    assert loco.loco_config_check(loco.Config(bits=1, **{k: v for k, v in good.items() if k != "bits"})) == loco.OK


def test_null_arguments_return_codes_without_a_device():
    L = loco.lib()
    assert L.loco_state_init(None, None, 0, None, 0, None) == loco.ERR_ARG
    h = C.c_void_p()
    assert L.loco_state_init(C.byref(h), None, 10, None, 0, None) == loco.ERR_ARG
    assert L.loco_state_reset(None, None) == loco.ERR_ARG
    assert L.loco_state_destroy(None) == loco.ERR_ARG
    assert L.loco_compensate_quantize_pack(None, None, None, 0, None) == loco.ERR_ARG
    assert L.loco_last_status(None, None, None, None) == loco.ERR_ARG
    assert L.loco_unpack_dequant_reduce(None, None, 1, 10, 0, 1, None, None) == loco.ERR_ARG
    assert loco.status_string(loco.ERR_ALIGN) == "LOCO_ERR_ALIGN"
    assert loco.status_string(0) == "LOCO_OK"

"""Host-side checks that need no GPU: the library builds for sm_100a, loads, and
exports every symbol the header declares; the binding's structs match the header's sizes."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2603_25702_b200.build import build
    return ctypes.CDLL(build())


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "s2d2.h")).read()
    names = set(re.findall(r"^(?:int|const char\*)\s+(s2d2_\w+)\s*\(", header, flags=re.M))
    assert len(names) >= 20
    for n in sorted(names):
        assert hasattr(lib, n), n
    from paper_2603_25702_b200.binding import EXPORTS
    assert set(EXPORTS) == names


def test_struct_sizes_match_header():
    from paper_2603_25702_b200 import binding as b
    assert ctypes.sizeof(b.ModelConfigC) == 13 * 4 + 3 * 4
    assert ctypes.sizeof(b.DecodeConfigC) == 13 * 4
    assert ctypes.sizeof(b.DraftStats) == 7 * 4 + 5 * 32 * 4
    assert ctypes.sizeof(b.StepResult) == 8 * 4 + 5 * 32 * 4
    assert ctypes.sizeof(b.Counters) == 9 * 8 + 33 * 8 + 4 * 8 + 9 * 8
    assert ctypes.sizeof(b.RoutePolicy) == 7 * 4


def test_create_without_gpu_fails_loudly(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    from paper_2603_25702_b200 import Engine, S2D2Error
    from s2d2_inputs import get_config
    with pytest.raises(S2D2Error):
        Engine(get_config("t_f32").model, block_size=4, max_batch=1, max_seq_len=32)


def test_oracle_and_product_do_not_import_each_other():
    pkg = os.path.join(ROOT, "paper_2603_25702_b200")
    for root, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                assert "oracle" not in open(os.path.join(root, f)).read().replace("oracle's", ""), f
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith(".py"):
            assert "paper_2603_25702_b200" not in open(os.path.join(ROOT, "oracle", f)).read(), f

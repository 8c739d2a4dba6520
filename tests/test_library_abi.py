"""The C-ABI library builds for sm_100a, loads without a GPU and exports every declared symbol."""
import ctypes
import os
import re

import pytest

from paper_2609_21264_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    path = build.build()
    return ctypes.CDLL(path)


def declared_functions():
    text = open(os.path.join(ROOT, "include", "fa.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"\b(fa_[a-z_]+)\s*\(", text)
    return sorted(set(names))


def test_header_declares_the_boundary():
    names = declared_functions()
    for must in ("fa_create", "fa_forward", "fa_destroy", "fa_last_status", "fa_strerror", "fa_forward_host"):
        assert must in names


def test_every_declared_symbol_is_exported(lib):
    for name in declared_functions():
        assert hasattr(lib, name), name


def test_binding_names_match_header():
    from paper_2609_21264_b200 import binding
    for name in declared_functions():
        assert hasattr(binding, name), name
        assert name in binding.EXPORTS


def test_strerror_and_null_handle_paths_need_no_gpu(lib):
    lib.fa_strerror.restype = ctypes.c_char_p
    seen = {lib.fa_strerror(i) for i in range(7)}
    assert len(seen) == 7 and b"success" in seen
    assert lib.fa_destroy(None) == 0
    lib.fa_launch_count.restype = ctypes.c_uint64
    assert lib.fa_launch_count(None) == 0
    assert lib.fa_create(None, None) == 1     # FA_ERR_INVALID_ARG: no out pointer


def test_create_without_device_fails_loudly():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    from paper_2609_21264_b200 import binding
    with pytest.raises(binding.FaError) as ei:
        binding.fa_create()
    assert ei.value.status == binding.FA_ERR_NO_DEVICE


def test_kv_tile_count_matches_visibility_rule():
    # host-side restatement of the causal loop bound, against enumeration of visible keys
    def kv_tiles(i0, rows, Sq, Sk, causal):
        last_key = Sk - 1
        if causal:
            last_row = min(i0 + rows - 1, Sq - 1)
            last_key = min(last_key, last_row + Sk - Sq)
        return 0 if last_key < 0 else last_key // 128 + 1
    for Sq, Sk in [(128, 128), (300, 300), (333, 200), (200, 333), (1, 500), (500, 1), (1024, 1024)]:
        for causal in (False, True):
            for i0 in range(0, Sq, 128):
                vis = [j for i in range(i0, min(i0 + 128, Sq)) for j in range(Sk)
                       if (not causal) or j <= i + Sk - Sq]
                want = 0 if not vis else max(vis) // 128 + 1
                assert kv_tiles(i0, 128, Sq, Sk, causal) == want


def test_flag_and_status_constants_match_the_header():
    """The binding's FA_FLAG_* / FA_* constants are the header's, name for name and value for value."""
    from paper_2609_21264_b200 import binding
    text = open(os.path.join(ROOT, "include", "fa.h")).read()
    flags = dict(re.findall(r"#define\s+(FA_FLAG_[A-Z_]+)\s+(\d+)u", text))
    assert len(flags) >= 8
    for name, value in flags.items():
        assert getattr(binding, name) == int(value), name
    values = [int(v) for v in flags.values()]
    assert len(set(values)) == len(values) and all(v & (v - 1) == 0 for v in values)     # distinct single bits
    for name in dir(binding):
        if name.startswith("FA_FLAG_"):
            assert name in flags, name


def test_plan_info_struct_matches_the_header():
    """fa_plan_info is read through ctypes: field order and types must follow the header's struct."""
    from paper_2609_21264_b200 import binding
    text = open(os.path.join(ROOT, "include", "fa.h")).read()
    body = re.search(r"typedef struct fa_plan_info \{(.*?)\} fa_plan_info;", text, flags=re.S).group(1)
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    fields = re.findall(r"(const char\*|int32_t|int64_t|double)\s+([a-z_]+(?:\s*,\s*[a-z_]+)*)\s*;", body)
    header = []
    for ctype, names in fields:
        for n in names.split(","):
            header.append((n.strip(), ctype))
    ctypes_of = {"const char*": ctypes.c_char_p, "int32_t": ctypes.c_int32, "int64_t": ctypes.c_int64, "double": ctypes.c_double}
    assert [(n, ctypes_of[t]) for n, t in header] == list(binding.fa_plan_info._fields_)

"""Host-only checks of the C ABI: the library loads, exports every declared symbol, and validates arguments."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    from paper_2512_19206_b200 import build
    build.build()
    from paper_2512_19206_b200 import binding as b
    return b


def test_library_exports_every_declared_symbol(binding):
    header = open(os.path.join(ROOT, "include", "mixkvq.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = sorted(set(re.findall(r"\b(mixkvq_[a-z_0-9]+)\s*\(", header)))
    assert len(declared) >= 12
    lib = C.CDLL(binding.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), name
    assert sorted(binding.EXPORTS) == declared


def test_header_is_plain_c_and_cpp(tmp_path):
    """include/mixkvq.h compiles by itself as C99 and as C++ (no CUDA or torch type in any signature), and the struct
    sizes the binding assumes are the compiler's."""
    import subprocess
    inc = os.path.join(ROOT, "include")
    src = ('#include "mixkvq.h"\n#include <stdio.h>\n'
           'int main(void) { printf("%zu %zu\\n", sizeof(mixkvq_config), sizeof(mixkvq_layout_desc)); return 0; }\n')
    for compiler, name, std in (("gcc", "t.c", "-std=c99"), ("g++", "t.cpp", "-std=c++14")):
        f = tmp_path / name
        f.write_text(src)
        exe = tmp_path / (name + ".out")
        subprocess.run([compiler, std, "-Wall", "-Werror", "-pedantic", "-I", inc, str(f), "-o", str(exe)], check=True)
        sizes = subprocess.run([str(exe)], capture_output=True, text=True, check=True).stdout.split()
        from paper_2512_19206_b200 import binding as b
        assert [int(x) for x in sizes] == [C.sizeof(b.Config), C.sizeof(b.LayoutDesc)]


def test_config_struct_matches_header(binding):
    assert C.sizeof(binding.Config) == 80          # 14 int32/float fields, one uint64, two budgets, sink length, pad
    assert C.sizeof(binding.LayoutDesc) == 13 * 8 + 4 * 4 + 2 * 8 + 2 * 4


def test_cache_bytes_and_argument_validation(binding):
    cfg = binding.make_config(2, 2, 8, 2, 1024)
    nbytes, ws = binding.cache_bytes(cfg)
    # per stream: 8 blocks of 12288 B, 32 KiB extras, 2 x 32 KiB residual, table, state
    assert nbytes > 2 * 4 * (8 * 12288 + 32768 + 65536)
    assert ws >= (148 * 8) * 8 * 130 * 4
    lib = binding.lib()
    for field, bad, code in [("head_dim", 64, -2), ("v_bits", 3, -2), ("group_size", 48, -2), ("residual_len", 100, -2),
                             ("residual_len", 512, -2), ("n_q_heads", 7, -1), ("batch", 0, -1), ("score_bits", 3, -2),
                             ("n_q_heads", 32, -2)]:
        c = binding.make_config(2, 2, 8, 2, 1024)
        setattr(c, field, bad)
        assert lib.mixkvq_cache_bytes(C.byref(c), None, None) == code, field
    c = binding.make_config(1, 1, 1, 1, 256, residual_len=64, group_size=32, block_layout=1)
    assert lib.mixkvq_cache_bytes(C.byref(c), None, None) == -2          # the tile layout needs R = 128
    c = binding.make_config(1, 1, 1, 1, 256, residual_len=64, group_size=128)
    assert lib.mixkvq_cache_bytes(C.byref(c), None, None) == -2          # R must be a multiple of G
    c = binding.make_config(1, 1, 1, 1, 256, block_layout=1, v_bits=4)
    assert lib.mixkvq_cache_bytes(C.byref(c), None, None) == -2          # 4-bit values: fragment layout only
    for field, bad in [("sink_len", 48), ("sink_len", 512), ("budget_bf16", 100), ("reserved", 1)]:
        c = binding.make_config(1, 1, 1, 1, 256, budget_u4=40)
        setattr(c, field, bad)
        assert lib.mixkvq_cache_bytes(C.byref(c), None, None) == -1, field
    assert lib.mixkvq_cache_bytes(None, None, None) == -1
    assert binding.status_string(-5) == "append exceeds max_tokens"
    assert binding.status_string(0) == "ok"


def test_null_handles_are_rejected(binding):
    lib = binding.lib()
    assert lib.mixkvq_quantize_append(None, 0, None, None, None, 1, None) == -1
    assert lib.mixkvq_decode_attention(None, 0, None, None, 1.0, None, 0, None) == -1
    assert lib.mixkvq_select_channels(None, 0, None, None, None) == -1
    assert lib.mixkvq_select_channels_raw(None, None, 1, 1, 1, 1, 1, 2, 1.0, 1.0, None, None, None) == -1
    assert lib.mixkvq_query_status(None, None, None) == -1
    assert lib.mixkvq_launch_count(None) == 0


def test_missing_library_fails_loudly(binding, monkeypatch):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", "/nonexistent/libmixkvq.so")
    with pytest.raises(RuntimeError, match="no fallback"):
        binding.lib()

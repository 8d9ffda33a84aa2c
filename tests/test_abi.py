"""The C-ABI library loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2502_20330_b200 import build
    return ctypes.CDLL(build.build())


def _declared():
    text = open(os.path.join(ROOT, "include", "rapid.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(rapid_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert "rapid_verify_attention" in names and "rapid_accept" in names and "rapid_verify_step" in names
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in rapid.h but not exported"


def test_binding_covers_the_header():
    from paper_2502_20330_b200 import binding
    assert sorted(binding.EXPORTS) == _declared()


def test_host_only_calls(lib):
    import paper_2502_20330_b200 as R
    assert R.version() == 100
    assert R.last_error() == ""
    assert R.attention_workspace_bytes(1, 32, 8, 128, 131072, 8) > 0
    assert R.attention_workspace_bytes(1, 32, 7, 128, 131072, 8) == 0     # Hq not a multiple of Hkv
    assert R.accept_workspace_bytes(8, 4, 152064) > 0
    assert R.accept_workspace_bytes(0, 4, 152064) == 0
    a = R.verify_step_host_arena_bytes(1, 8, 2, 64, 4096, 4, 4096)
    assert a > 2 * 2 * 4096 * 64 * 2


def test_retrieval_budget_rule():
    """Section 3.1, RAG set-up: max(4,096 tokens, context / 24) in chunks of 512 (host arithmetic of the library)."""
    import paper_2502_20330_b200 as R
    assert R.rapid_retrieval_budget_chunks(131072) == 10      # 131072/24 = 5461 tokens -> 10 chunks of 512
    assert R.rapid_retrieval_budget_chunks(32768) == 8        # the 4096-token floor
    assert R.rapid_retrieval_budget_chunks(1_000_000) == 81
    assert R.rapid_retrieval_budget_chunks(0) == 8
    with pytest.raises(ValueError):
        R.rapid_retrieval_budget_chunks(-1)
    with pytest.raises(ValueError):
        R.rapid_retrieval_budget_chunks(1000, chunk_tokens=0)


def test_struct_layouts_match_the_header():
    from paper_2502_20330_b200 import binding
    assert ctypes.sizeof(binding._AttnShape) == 48
    assert ctypes.sizeof(binding._AttnParams) == 72
    assert ctypes.sizeof(binding._AcceptShape) == 32
    assert ctypes.sizeof(binding._AcceptParams) == 40
    assert ctypes.sizeof(binding._PagedKv) == 40


def test_struct_layouts_match_what_the_c_compiler_sees(tmp_path):
    """sizeof and the offset of the last field of every struct, as gcc lays the header out."""
    import subprocess
    from paper_2502_20330_b200 import binding
    src = tmp_path / "layout.c"
    src.write_text(
        '#include <stdio.h>\n#include <stddef.h>\n#include "rapid.h"\n'
        'int main(void) {\n'
        '  printf("%zu %zu\\n", sizeof(rapid_attn_shape), offsetof(rapid_attn_shape, kv_stride_l));\n'
        '  printf("%zu %zu\\n", sizeof(rapid_attn_params), offsetof(rapid_attn_params, kv_settled));\n'
        '  printf("%zu %zu\\n", sizeof(rapid_accept_shape), offsetof(rapid_accept_shape, draft_row_stride));\n'
        '  printf("%zu %zu\\n", sizeof(rapid_accept_params), offsetof(rapid_accept_params, draft_logq));\n'
        '  printf("%zu %zu\\n", sizeof(rapid_paged_kv), offsetof(rapid_paged_kv, stride_l));\n'
        '  return 0;\n}\n')
    exe = tmp_path / "layout"
    subprocess.run(["gcc", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)], check=True)
    got = [tuple(int(x) for x in line.split()) for line in subprocess.run([str(exe)], check=True, capture_output=True,
                                                                          text=True).stdout.splitlines()]
    want = [(ctypes.sizeof(c), getattr(c, f).offset) for c, f in (
        (binding._AttnShape, "kv_stride_l"), (binding._AttnParams, "kv_settled"),
        (binding._AcceptShape, "draft_row_stride"), (binding._AcceptParams, "draft_logq"),
        (binding._PagedKv, "stride_l"))]
    assert got == want


def test_product_does_not_touch_the_oracle():
    pkg = os.path.join(ROOT, "paper_2502_20330_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src, f"{f} mentions the oracle"

"""Host-side checks that need no GPU: the C-ABI library loads and exports every entry point the
public header declares, and the ctypes mirrors of the structs have the C sizes."""
import ctypes
import os
import re
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "tasc.h")


@pytest.fixture(scope="module")
def lib_path():
    sys.path.insert(0, ROOT)
    from paper_2602_24174_b200 import build
    return build.build()


def declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(tasc_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_named_entry_points():
    names = declared_functions()
    for must in ("tasc_drafter_build", "tasc_draft", "tasc_verify_step", "tasc_generate"):
        assert must in names


def test_library_exports_every_declared_symbol(lib_path):
    lib = ctypes.CDLL(lib_path)
    for name in declared_functions():
        assert hasattr(lib, name), f"{name} is declared in tasc.h but not exported"


def test_struct_sizes_match_c(lib_path, tmp_path):
    src = tmp_path / "sizes.c"
    src.write_text('#include <stdio.h>\n#include "tasc.h"\nint main(void){printf("%zu %zu %zu %zu %zu %zu %zu %zu %zu\\n",'
                   "sizeof(tasc_ngram_entry),sizeof(tasc_model_desc),sizeof(tasc_weights),sizeof(tasc_kv),"
                   "sizeof(tasc_seqs),sizeof(tasc_draft_params),sizeof(tasc_stats),sizeof(tasc_status),"
                   "sizeof(tasc_corpus_statistics));return 0;}\n")
    exe = tmp_path / "sizes"
    subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)])
    sizes = list(map(int, subprocess.check_output([str(exe)]).split()))
    from paper_2602_24174_b200 import binding as b
    mirrors = [b.NgramEntry, b.ModelDesc, b.Weights, b.Kv, b.Seqs, b.DraftParams, b.Stats, ctypes.c_int32, b.CorpusStatistics]
    assert sizes == [ctypes.sizeof(m) for m in mirrors]


def test_status_strings(lib_path):
    from paper_2602_24174_b200 import binding as b
    assert b.lib.tasc_status_string(0) == b"ok"
    assert b"KV" in b.lib.tasc_status_string(b.ENOKV)


def test_argument_checks_need_no_device(lib_path):
    from paper_2602_24174_b200 import binding as b
    h = ctypes.c_void_p()
    assert b.lib.tasc_drafter_build(None, None, 0, 3, 1, 10, None, ctypes.byref(h)) == b.EINVAL
    assert b.lib.tasc_model_create(None, None, ctypes.byref(h)) == b.EINVAL
    st = b.CorpusStatistics()
    assert b.lib.tasc_corpus_stats(None, None, 0, 10, 4, 5, None, ctypes.byref(st)) == b.EINVAL
    assert b.lib.tasc_gemm_workspace_bytes(0, 1, 1) == 0
    assert b.lib.tasc_gemm_workspace_bytes(6, 1152, 896) >= 6 * 1152 * 4

"""Host-side checks that need no GPU: the library loads, exports every symbol the
header declares, and rejects bad descriptions before touching CUDA."""
import ctypes
import os
import re

import pytest

from paper_2512_16843_b200 import binding as L

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "llmcache.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(llmcache_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(L.LIB_PATH)
    names = declared_symbols()
    assert len(names) >= 14
    for name in names:
        assert hasattr(lib, name), name
    assert sorted(L.EXPORTS) == names


def test_abi_version_and_strerror():
    assert L.llmcache_abi_version() == 2
    assert L.strerror(0) == "ok" and "argument" in L.strerror(L.ERR_ARG)


def test_struct_layout_matches_header_order():
    assert ctypes.sizeof(L.BankDesc) == 17 * 4 + 4 + 4 * 8      # 17 words + padding + 3 pointers + size_t
    assert ctypes.sizeof(L.ProbeIO) == 11 * 8
    assert ctypes.sizeof(L.Stats) == 11 * 8


@pytest.mark.parametrize("kw,status", [
    (dict(capacity=0), L.ERR_SHAPE),
    (dict(d_model=100), L.ERR_SHAPE),
    (dict(fp_dim=100), L.ERR_SHAPE),
    (dict(fp_dim=128), L.ERR_SHAPE),          # no projection: k must equal d
    (dict(hidden_dtype=7), L.ERR_ARG),
    (dict(policy=9), L.ERR_ARG),
    (dict(act_rows=9999), L.ERR_SHAPE),
    (dict(max_batch=0), L.ERR_SHAPE),
    (dict(tau=float("nan")), L.ERR_ARG),
])
def test_bad_descriptions_are_rejected_on_the_host(kw, status):
    base = dict(capacity=16, seq_len=8, d_model=64, fp_dim=64, max_batch=4)
    base.update(kw)
    with pytest.raises(L.LLMCacheError) as e:
        L.llmcache_bank_bytes(L.make_desc(**base))
    assert e.value.status == status


def test_bank_bytes_counts_the_activation_store():
    d = L.make_desc(capacity=2048, seq_len=384, d_model=768, fp_dim=768, max_batch=256)
    assert L.llmcache_bank_bytes(d) >= 2048 * 384 * 768 * 2
    d.struct_size = 8
    with pytest.raises(L.LLMCacheError):
        L.llmcache_bank_bytes(d)


def test_null_handles_are_rejected():
    lib = L.lib()
    assert lib.llmcache_bank_destroy(None) == L.ERR_ARG
    assert lib.llmcache_bank_status(None) == L.ERR_ARG
    assert lib.llmcache_evict(None, 0, None, 0, None, None) == L.ERR_ARG


def test_no_cpu_fallback_without_a_device():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    with pytest.raises(L.LLMCacheError) as e:
        L.llmcache_bank_create(L.make_desc(capacity=16, seq_len=8, d_model=64, fp_dim=64, max_batch=4))
    assert e.value.status == L.ERR_CUDA


def test_header_is_plain_c(tmp_path):
    """The boundary is a C ABI: the header must compile as C99 on its own, and a C program must link against the
    library using nothing but that header."""
    import shutil
    import subprocess
    gcc = shutil.which("gcc")
    if gcc is None:
        pytest.skip("no C compiler")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    src = tmp_path / "use_header.c"
    src.write_text(
        '#include "llmcache.h"\n'
        "#include <stdio.h>\n"
        "int main(void) {\n"
        "  llmcache_bank_desc d = {0};\n"
        "  size_t bytes = 0;\n"
        "  d.struct_size = (uint32_t)sizeof d; d.capacity = 4; d.seq_len = 2; d.d_model = 64; d.fp_dim = 64;\n"
        "  d.max_batch = 2; d.hidden_dtype = LLMCACHE_BF16; d.store_act = 1; d.tau = 0.9f;\n"
        "  if (llmcache_abi_version() != LLMCACHE_ABI_VERSION) return 2;\n"
        "  if (llmcache_bank_bytes(&d, &bytes) != LLMCACHE_OK || bytes == 0) return 3;\n"
        '  printf("%s %zu\\n", llmcache_strerror(LLMCACHE_ERR_SHAPE), bytes);\n'
        "  return 0;\n"
        "}\n")
    exe = tmp_path / "use_header"
    lib_dir = os.path.dirname(L.LIB_PATH)
    r = subprocess.run([gcc, "-std=c99", "-Wall", "-Werror", "-pedantic", "-I", os.path.join(root, "include"), str(src),
                        "-o", str(exe), "-L", lib_dir, "-l:libllmcache.so", "-Wl,-rpath," + lib_dir],
                       capture_output=True, text=True)
    assert r.returncode == 0, r.stderr
    r = subprocess.run([str(exe)], capture_output=True, text=True)
    assert r.returncode == 0, (r.returncode, r.stdout, r.stderr)
    assert "shape" in r.stdout

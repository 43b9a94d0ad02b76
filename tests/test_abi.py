"""The C-ABI library: loads without a GPU, exports every declared symbol, validates before touching CUDA."""
import ctypes
import os
import re

import pytest

import __graft_entry__ as entry
from paper_2503_14985_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    entry.build()
    return binding.load()


def test_header_symbols_are_exported(lib):
    header = open(os.path.join(ROOT, "include", "mlt.h")).read()
    declared = set(re.findall(r"^(?:int|size_t|const char\*)\s+(mlt_[a-z_0-9]+)\s*\(", header, flags=re.M))
    assert declared >= set(binding.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), f"{name} declared in mlt.h but not exported"


def test_version_and_status_strings(lib):
    assert binding.version() >= 100
    texts = {binding.status_string(i) for i in range(9)}
    assert len(texts) == 9 and "unknown status" not in texts
    assert binding.status_string(99) == "unknown status"


def test_validation_precedes_cuda(lib):
    # none of these may reach a CUDA call (there may be no GPU here): the status must be the validation one
    assert binding.gemm_raw(0, 0, 0, -1, 1, 1, 8, 8, 8) == 1
    assert binding.gemm_raw(0, 0, 0, 0, 8, 8, 8, 8, 8) == 0
    assert binding.gemm_raw(16, 16, 0, 4, 4, 4, 8, 8, 8) == 1
    assert binding.gemm_raw(16, 16, 16, 4, 4, 4, 8, 8, 2) == 1
    assert binding.gemm_raw(16, 16, 16, 4, 4, 4, 8, 8, 12) == 3
    assert binding.gemm_raw(16, 16, 18, 4, 4, 4, 8, 8, 8) == 3
    assert binding.mha_fwd_raw(16, 16, 16, 16, 0, 1, 1, 8, 8, 80, 0, 1.0) == 2
    assert binding.mha_fwd_raw(16, 16, 16, 16, 0, 1, 1, 9, 8, 64, 1, 1.0) == 1
    assert binding.mha_fwd_raw(16, 16, 16, 16, 0, 0, 4, 9, 8, 64, 0, 1.0) == 0
    assert binding.mha_fwd_raw(16, 16, 16, 16, 0, 1, 1, 8, 8, 64, 0, float("nan")) == 1
    pa = binding.paged_attn_decode_raw
    assert pa(16, 16, 16, 16, 16, 16, 0, 0, 8, 8, 128, 16, 4, 10, 1.0) == 0          # no sequences
    assert pa(16, 16, 16, 16, 16, 16, 0, 2, 8, 3, 128, 16, 4, 10, 1.0) == 1          # H not a multiple of H_kv
    assert pa(16, 16, 16, 16, 16, 16, 0, 2, 8, 8, 96, 16, 4, 10, 1.0) == 2           # head dimension
    assert pa(16, 16, 16, 16, 16, 16, 0, 2, 8, 8, 128, 12, 4, 10, 1.0) == 2          # block size
    assert pa(16, 16, 16, 16, 16, 16, 0, 2, 24, 2, 128, 16, 4, 10, 1.0) == 2         # 12 query heads per KV head
    assert pa(16, 18, 16, 16, 16, 16, 0, 2, 8, 8, 128, 16, 4, 10, 1.0) == 3          # misaligned cache
    assert pa(16, 16, 16, 0, 16, 16, 0, 2, 8, 8, 128, 16, 4, 10, 1.0) == 1           # NULL block table
    assert binding.paged_attn_workspace_bytes(64, 32, 128) == 64 * 32 * 32 * (128 * 4 + 8)


def test_product_does_not_import_oracle():
    pkg = os.path.join(ROOT, "paper_2503_14985_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in text and "from oracle" not in text and "oracle/" not in text, f


def test_build_refuses_an_attention_kernel_below_its_register_budget():
    # The attention kernel hands registers from its idle warps to its softmax warps; a build whose launch allocation
    # is smaller than that hand-over needs must never be launched (the increase would wait for ever), so the build
    # step reads the compiler's report and fails.  Checked here on report texts, no GPU involved.
    from paper_2503_14985_b200 import build
    ok = ("ptxas info    : Compiling entry function '_ZN3mlt14mha_fwd_kernelILi128EEEv' for 'sm_100a'\n"
          "ptxas info    : Used 168 registers, used 1 barriers\n"
          "ptxas info    : Compiling entry function '_ZN3mlt9other_fooEv' for 'sm_100a'\n"
          "ptxas info    : Used 32 registers, used 0 barriers\n")
    assert build.check_mha_registers(ok) == {"_ZN3mlt14mha_fwd_kernelILi128EEEv": 168}
    with pytest.raises(RuntimeError):
        build.check_mha_registers(ok.replace("Used 168", "Used 160"))
    assert build.check_mha_registers("nothing here") == {}

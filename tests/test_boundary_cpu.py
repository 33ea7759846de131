"""The C-ABI library builds, loads without a GPU, and exports every symbol the header declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "dlm.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dlm_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_four_hot_path_calls():
    names = declared_functions()
    for required in ("dlm_kv_cache_commit", "dlm_freecache_attn_step", "dlm_unmask_select", "dlm_guided_accept"):
        assert required in names


def test_library_exports_every_declared_symbol():
    from paper_2505_21467_b200 import build
    lib = ctypes.CDLL(build.build())
    for name in declared_functions():
        assert hasattr(lib, name), f"{name} is declared in dlm.h but not exported"


def test_binding_has_the_same_names_and_fails_loudly_without_a_gpu():
    import torch
    import paper_2505_21467_b200 as dlm
    for name in declared_functions():
        assert hasattr(dlm, name), f"binding lacks {name}"
    assert dlm.dlm_strerror(0) == "ok" and "index" in dlm.dlm_strerror(dlm.DLM_ERR_INDEX)
    if not torch.cuda.is_available():
        try:
            dlm.dlm_create(0)
        except dlm.DlmError as e:
            assert e.code == dlm.DLM_ERR_CUDA
        else:
            raise AssertionError("dlm_create must fail without a CUDA device")


def test_product_package_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_2505_21467_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src, f"{f} mentions the oracle"


def test_build_checks_the_attention_kernels_register_count():
    """The attention kernel's setmaxnreg split balances only at 168 registers per thread at launch: the build reads
    ptxas's log and refuses any other number (a run-time DLM_ERR_UNSUPPORTED otherwise)."""
    from paper_2505_21467_b200 import build as b
    ok = ("ptxas info    : Compiling entry function '_ZN3foo22attn_step_sm100_kernelILi128ELi256ELb0EEEv' for 'sm_100a'\n"
          "ptxas info    : Used 168 registers, used 1 barriers\n"
          "ptxas info    : Compiling entry function 'other_kernel' for 'sm_100a'\nptxas info    : Used 40 registers\n")
    b.check_attention_registers(ok)
    with pytest.raises(RuntimeError):
        b.check_attention_registers(ok.replace("Used 168", "Used 160"))
    with pytest.raises(RuntimeError):
        b.check_attention_registers("ptxas info    : Compiling entry function 'other_kernel' for 'sm_100a'\nptxas info    : Used 40 registers\n")

"""Host-side checks that need no GPU: the library loads and exports what the header declares."""
import ctypes as C

import pytest
import torch

import paper_2411_03786_b200 as ngs


def test_library_loads_and_exports_every_declared_symbol():
    lib = ngs.load_library()
    names = ngs.declared_symbols()
    assert {"spec_init", "spec_destroy", "spec_get_status", "spec_last_error", "build_model_ngram_tables",
            "draft_context_ngrams", "verify_lmhead_argmax", "accept_and_commit", "spec_debug_logits"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in include/ngram_spec.h but not exported"


def test_argument_errors_are_reported_without_touching_a_gpu():
    lib = ngs.load_library()
    h = C.c_void_p()
    assert lib.spec_init(C.byref(h), None, None, 1, 8, 8, 0, None) == -1
    assert b"NULL" in lib.spec_last_error(None)
    assert lib.spec_init(C.byref(h), C.c_void_p(16), C.c_void_p(32), 1, 8, 12, 0, None) == -1   # d % 8 != 0
    assert lib.spec_init(C.byref(h), C.c_void_p(8), C.c_void_p(32), 1, 8, 8, 0, None) == -1     # misaligned
    assert lib.verify_lmhead_argmax(None, None, 1, None, None, None) == -1
    assert lib.accept_and_commit(None, None, None, None, 1, 1, 1, None, None, 4, None, None, None, None) == -1


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-GPU failure mode")
def test_no_cpu_fallback():
    lib = ngs.load_library()
    h = C.c_void_p()
    rc = lib.spec_init(C.byref(h), C.c_void_p(256), C.c_void_p(512), 1, 8, 8, 0, None)
    assert rc == -3 and not h.value
    with pytest.raises(ngs.SpecError):
        ngs.SpecContext(torch.zeros(8, 8, dtype=torch.bfloat16), torch.zeros(8, 8, dtype=torch.bfloat16))

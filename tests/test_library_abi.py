"""The C-ABI library loads and exports every symbol that include/eventgrad.h declares.
No compute call is made here (no GPU needed)."""
import ctypes
import os
import re

from paper_2103_07454_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "eventgrad.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(eg_[a-z_0-9]+)\s*\(", text)))


def test_header_symbols_are_exported():
    lib = ctypes.CDLL(build.build())
    names = declared_functions()
    assert "eg_create" in names and "eg_step" in names and "eg_stats" in names
    for name in names:
        assert hasattr(lib, name), f"{name} declared in eventgrad.h but not exported"


def test_binding_covers_the_header():
    assert sorted(binding.EXPORTS) == declared_functions()


def test_status_strings():
    lib = binding.load_library()
    assert lib.eg_strerror(0) == b"ok"
    assert lib.eg_strerror(1) == b"invalid argument"
    assert lib.eg_last_cuda_error(None) == 0


def test_error_word_decoding():
    """What the synchronising calls make of the device-side error word: a bounded wait that ran
    out is a time-out, a failed index check or a misplaced Top-K entry an internal error."""
    lib = binding.load_library()
    assert lib.eg_status_of_error_word(0) == 0
    assert lib.eg_status_of_error_word(2) == 6 and lib.eg_status_of_error_word(4) == 6
    assert lib.eg_status_of_error_word(8) == 5 and lib.eg_status_of_error_word(8 | 4 | 2) == 5
    assert lib.eg_strerror(5) == b"timeout"
    assert lib.eg_debug_build() in (0, 1)


def test_create_rejects_bad_arguments_before_touching_the_device():
    lib = binding.load_library()
    h = ctypes.c_void_p()
    thr = binding.ThresholdParams(0, 1.0, 1, 0.0, 0.0, 1)
    numel = (ctypes.c_int64 * 2)(4, 0)
    assert lib.eg_create(ctypes.byref(h), 0, 4, numel, 2, ctypes.byref(thr), None) == 1   # empty tensor
    numel = (ctypes.c_int64 * 2)(4, 5)
    assert lib.eg_create(ctypes.byref(h), 8, 4, numel, 2, ctypes.byref(thr), None) == 1   # topology
    assert lib.eg_create(ctypes.byref(h), -1, 4, numel, 2, ctypes.byref(thr), None) == 1
    assert lib.eg_create(ctypes.byref(h), 0, 0, numel, 2, ctypes.byref(thr), None) == 1   # P
    thr.history_len = 0
    assert lib.eg_create(ctypes.byref(h), 0, 4, numel, 2, ctypes.byref(thr), None) == 1   # H
    assert not h.value

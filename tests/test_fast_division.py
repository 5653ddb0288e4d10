"""CPU proof that the reciprocal-based division of the kernels is the IEEE quotient for every
bfloat16 operand pair in the range where the kernels use it (Eq. 2 must be exact because the
4-bit codes are compared bit for bit)."""
import ctypes
import os
import subprocess

import pytest

HERE = os.path.dirname(os.path.abspath(__file__))


@pytest.fixture(scope="module")
def lib(tmp_path_factory):
    so = str(tmp_path_factory.mktemp("fd") / "fd.so")
    src = os.path.join(HERE, "helpers", "fast_division_check.c")
    subprocess.run(["gcc", "-O2", "-std=c11", "-fno-fast-math", "-ffp-contract=off", "-shared", "-fPIC",
                    src, "-o", so, "-lm"], check=True)
    L = ctypes.CDLL(so)
    L.fast_division_mismatches.restype = ctypes.c_long
    L.truncated_sequence_mismatches.restype = ctypes.c_long
    return L


def test_sequence_equals_ieee_division_for_all_bf16_pairs(lib):
    checked = ctypes.c_long(0)
    # quotients down to 2^-41: far above the 2^-100 guard below which the kernels re-divide
    bad = lib.fast_division_mismatches(40, ctypes.byref(checked))
    assert checked.value > 300_000_000
    assert bad == 0


def test_the_sweep_catches_a_wrong_sequence(lib):
    checked = ctypes.c_long(0)
    bad = lib.truncated_sequence_mismatches(ctypes.byref(checked))
    assert checked.value == 128 * 128 and bad > 0

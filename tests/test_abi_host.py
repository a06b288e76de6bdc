"""Host-only checks of the C-ABI library: it loads, exports every declared symbol, and its
host logic (dyadic multipliers, argument validation) behaves -- no GPU needed."""
import ctypes as C
import math
import random
import re
from fractions import Fraction
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def lib():
    from paper_2101_01321_b200 import build, binding
    build.build()
    return binding.lib()


def test_every_declared_symbol_is_exported(lib):
    header = (ROOT / "include" / "ibert.h").read_text()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    names = re.findall(r"\b(ibert_[a-z0-9_]+)\s*\(", header)
    assert len(set(names)) >= 14
    for n in set(names):
        assert hasattr(lib, n), n


def test_strerror_covers_all_codes(lib):
    for code in range(0, -9, -1):
        assert lib.ibert_strerror(code).decode() not in ("", "unknown error")
    assert lib.ibert_strerror(-99).decode() == "unknown error"


def test_dyadic_from_double_is_nearest_multiplier(lib):
    from paper_2101_01321_b200.binding import ibert_dyadic_from_double, IbertError
    rnd = random.Random(7)
    for _ in range(3000):
        m = math.ldexp(rnd.uniform(0.5, 1.0), rnd.randint(-40, 30)) * rnd.choice((-1, 1))
        b, c = ibert_dyadic_from_double(m)
        assert 0 <= c <= 31 and abs(b) < 2 ** 31
        assert abs(Fraction(b, 2 ** c) - Fraction(m)) <= Fraction(1, 2 ** (c + 1))
    assert ibert_dyadic_from_double(0.0) == (0, 0)
    assert ibert_dyadic_from_double(1.0) == (2 ** 30, 30)
    assert ibert_dyadic_from_double(2.0 ** 30) == (2 ** 30, 0)
    with pytest.raises(IbertError):
        ibert_dyadic_from_double(2.0 ** 31)
    with pytest.raises(IbertError):
        ibert_dyadic_from_double(float("inf"))


def test_dyadic_matches_the_oracle_bit_for_bit(lib):
    import oracle
    from paper_2101_01321_b200.binding import ibert_dyadic_from_double
    rnd = random.Random(8)
    for _ in range(3000):
        m = math.ldexp(rnd.uniform(0.5, 1.0), rnd.randint(-45, 30)) * rnd.choice((-1, 1))
        assert ibert_dyadic_from_double(m) == oracle.dyadic(m)


def test_calls_reject_bad_arguments_before_touching_a_device(lib):
    null = C.c_void_p()
    assert lib.ibert_gelu_i(None, None, 1e-3, 4, 0.03, None, None) == -1
    assert lib.ibert_softmax_i(None, None, 1e-3, 1, 8, 255, None, None) == -1
    assert lib.ibert_layernorm_i(None, None, 1e-3, None, 0.0, None, None, 1, 8, 0.02, None, None) == -1
    assert lib.ibert_linear_i8(None, None, 1.0, None, None, None, 1, 16, 16, 0, 1.0, None, None) == -1
    assert lib.ibert_attention_i8(None, None, 1, 8, 64, 1, 1.0, 1.0, 1.0, 1.0, 255, None, None) == -1
    assert lib.ibert_encoder_layer(None, None, None, 1, 8, None, None) == -1
    assert lib.ibert_layer_create(None, None, C.byref(null)) == -1
    assert lib.ibert_destroy(None) == -1
    assert lib.ibert_last_status(None) == -1
    assert lib.ibert_create(None, 0, None) == -1


def test_create_fails_cleanly_without_a_usable_device(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    h = C.c_void_p()
    assert lib.ibert_create(C.byref(h), 0, None) == -6      # IBERT_ERR_CUDA, no fallback
    assert not h.value


def test_exp_division_by_multiplication_is_exact_for_every_distance(lib):
    # host emulation of the kernels' multiply-high division by q_ln2, all d in [0, 31 q_ln2]
    import oracle
    rnd = random.Random(9)
    scales = [0.69, 0.5, 0.3, 0.1, 1e-2, 1e-3, 4.5e-5, 3.8e-5, 2e-5, 1e-8, 4.13e-5, 8.2e-5, 8.3e-5]
    scales += [math.exp(rnd.uniform(math.log(1e-9), math.log(0.69))) for _ in range(300)]
    seen = set()
    for S in scales:
        q = C.c_int32()
        assert lib.ibert_selftest_exp_division(S, C.byref(q)) == 0, S
        assert q.value == oracle.exp_consts(S)["q_ln2"]
        seen.add(q.value.bit_length())
    assert len(seen) >= 12                     # divisors of many sizes were exercised
    assert lib.ibert_selftest_exp_division(0.7, None) == -3

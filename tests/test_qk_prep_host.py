"""Argument checks of `clear_qk_norm_rope` and the host arithmetic of `clear_log_scale_factor`, through the raw
C symbols.  Every call here is refused before any CUDA call is made, so no GPU is needed (the pointers are
never dereferenced)."""
import ctypes
import math

import pytest

from paper_2412_16112_b200 import binding as clear

FAKE = 0x10000  # 16-byte aligned, never touched


def _call(q=FAKE, k=FAKE, qo=FAKE, ko=FAKE, gq=None, gk=None, B=1, H=2, gh=4, gw=4, T=1, d=128, dtype=clear.BF16,
          axes=(16, 56, 56), theta=10000.0, ntk=1.0, eps=1e-6, qf=1.0):
    return clear.load().clear_qk_norm_rope(q, k, qo, ko, gq, gk, B, H, gh, gw, T, d, dtype, axes[0], axes[1], axes[2],
                                           theta, ntk, eps, qf, None)


@pytest.mark.parametrize("kw", [
    dict(B=0), dict(H=-1), dict(gh=0), dict(gw=0), dict(T=-1), dict(dtype=7),
    dict(axes=(15, 57, 56)),            # odd group sizes
    dict(axes=(16, 56, 54)),            # groups do not cover the head
    dict(axes=(-2, 66, 64)),
    dict(theta=0.0), dict(theta=float("inf")), dict(ntk=0.0), dict(ntk=float("nan")),
    dict(eps=-1e-6), dict(eps=float("nan")), dict(qf=float("inf")),
    dict(q=None), dict(ko=None),
])
def test_invalid_arguments_are_refused(kw):
    assert _call(**kw) == clear.ERR_INVALID_ARG


def test_unsupported_and_misaligned():
    assert _call(d=96, axes=(16, 40, 40)) == clear.ERR_UNSUPPORTED
    assert _call(k=FAKE + 8) == clear.ERR_MISALIGNED
    assert _call(gq=FAKE + 2) == clear.ERR_MISALIGNED


def test_log_scale_factor_host_arithmetic():
    f = clear.clear_log_scale_factor
    assert f(4608, 4608) == 1.0
    assert f(4096 ** 2, 4096) == pytest.approx(math.sqrt(2.0), rel=1e-6)
    assert f(16896, 4608) == pytest.approx(math.sqrt(math.log(16896) / math.log(4608)), rel=1e-6)
    assert f(1, 4608) == 1.0 and f(4608, 0) == 1.0

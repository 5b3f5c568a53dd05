"""The C-ABI library loads, exports every symbol the header declares, and rejects
host-detectable argument errors before touching the device (runs without a GPU)."""
import ctypes as C
import os
import re

import pytest

import paper_2606_12370_b200 as P
from paper_2606_12370_b200 import build as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    B.build()
    return P.load_library()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "bebop.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(bebop_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert {"bebop_verify", "bebop_tv", "bebop_greedy_verify", "bebop_workspace_bytes",
            "bebop_status_string"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_workspace_bytes_is_pure_and_monotone(lib):
    assert P.bebop_workspace_bytes(0, 3, 1024, 0) == 0
    assert P.bebop_workspace_bytes(4, 0, 1024, 0) == 0
    assert P.bebop_workspace_bytes(4, 33, 1024, 0) == 0
    assert P.bebop_workspace_bytes(4, 3, 1024, 7) == 0
    a = P.bebop_workspace_bytes(4, 3, 1024, 0)
    b = P.bebop_workspace_bytes(256, 3, 151936, 1)
    assert 0 < a and a % 256 == 0 and b % 256 == 0 and b >= a


def test_status_strings(lib):
    seen = {P.bebop_status_string(i) for i in range(9)}
    assert len(seen) == 9 and P.bebop_status_string(0) == "ok"


def _verify(lib, **kw):
    fake = 0x10000   # never dereferenced: every case below fails a host check first
    a = dict(target=fake, ldt=1024, draft=fake, ldd=1024, tok=fake, dl=None, temp=None, tall=1.0,
             ua=fake, uf=fake, B=4, K=3, V=1024, dt=0, acc=fake, out=fake, tv=None, pd=None, qd=None,
             st=None, ws=fake, wsb=1 << 30, stream=None)
    a.update(kw)
    return lib.bebop_verify(a["target"], a["ldt"], a["draft"], a["ldd"], a["tok"], a["dl"], a["temp"],
                            a["tall"], a["ua"], a["uf"], a["B"], a["K"], a["V"], a["dt"], a["acc"],
                            a["out"], a["tv"], a["pd"], a["qd"], a["st"], a["ws"], a["wsb"], a["stream"])


def test_host_validation_order(lib):
    assert _verify(lib, B=0) == 2
    assert _verify(lib, K=33) == 2
    assert _verify(lib, dt=5) == 3
    assert _verify(lib, target=None) == 1
    assert _verify(lib, tok=None) == 1
    assert _verify(lib, acc=None) == 1
    assert _verify(lib, ws=None) == 1
    assert _verify(lib, ldt=1000) == 2            # ld < V
    assert _verify(lib, V=1022, ldt=1022, ldd=1022) == 4   # 1022 * 4 bytes is not a multiple of 16
    assert _verify(lib, target=0x10004) == 4
    assert _verify(lib, tall=0.0) == 6
    assert _verify(lib, tall=float("nan")) == 6
    assert _verify(lib, wsb=16) == 5
    assert _verify(lib, ws=0x10010) == 4
    # greedy and tv share the checks
    fake = 0x10000
    assert lib.bebop_tv(fake, 512, fake, 512, None, 1.0, 0, 512, 0, fake, None, None, fake, 1 << 20, None) == 2
    assert lib.bebop_tv(fake, 512, fake, 512, None, 1.0, 4, 512, 0, None, None, None, fake, 1 << 20, None) == 1
    assert lib.bebop_greedy_verify(fake, 512, None, None, 4, 3, 512, 0, fake, fake, None, fake, 1 << 20, None) == 1
    assert lib.bebop_greedy_verify(fake, 100, fake, None, 4, 3, 512, 0, fake, fake, None, fake, 1 << 20, None) == 2


def test_missing_library_fails_loudly(monkeypatch):
    from paper_2606_12370_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_LIB_PATH", "/nonexistent/libbebop.so")
    with pytest.raises(ImportError):
        binding.load_library()

"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every
symbol the public header declares, and rejects bad arguments before touching CUDA."""
import ctypes
import os
import re

import pytest

from paper_2608_00867_b200 import binding as nb
from paper_2608_00867_b200 import build as nbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built_library():
    nbuild.build()


def declared_functions():
    """Functions declared by the public header(s) and by the internal header of the test hooks."""
    headers = [os.path.join(ROOT, "include", fn) for fn in os.listdir(os.path.join(ROOT, "include")) if fn.endswith(".h")]
    headers.append(os.path.join(ROOT, "paper_2608_00867_b200", "csrc", "nuna_debug.h"))
    names = set()
    for path in headers:
        text = open(path).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names |= set(re.findall(r"\b(nuna_[a-z0-9_]+)\s*\(", text))
    return sorted(names)


def test_no_undeclared_exports():
    """Every nuna_* symbol the library exports is declared in the public header or in the debug header."""
    import subprocess
    out = subprocess.run(["nm", "-D", "--defined-only", nb._LIB_PATH], capture_output=True, text=True, check=True).stdout
    exported = {ln.split()[-1] for ln in out.splitlines() if ln.split() and ln.split()[-1].startswith("nuna_")}
    assert exported <= set(declared_functions()), exported - set(declared_functions())


def test_every_declared_symbol_is_exported():
    names = declared_functions()
    assert {"nuna_allreduce_oneshot", "nuna_allreduce_twoshot", "nuna_reduce_scatter", "nuna_allgather"} <= set(names)
    L = nb.lib()
    for name in names:
        assert hasattr(L, name), f"{name} declared in include/ but not exported"


def test_status_strings():
    assert nb.status_string(nb.NUNA_OK) == "ok"
    seen = {nb.status_string(s) for s in range(10)}
    assert len(seen) == 10 and "unknown status" not in seen
    assert nb.status_string(1234) == "unknown status"


def test_validation_happens_before_any_cuda_call():
    A = 1 << 20          # fake, aligned "device" addresses: validation never dereferences them
    ok_src, ok_dst = [A, A + 4096], [A + 8192, A + 12288]
    call = lambda *a, **k: nb.nuna_allreduce_oneshot(*a, stream=0, check=False, **k)
    assert call([], [], 0, nranks=0) == nb.NUNA_ERR_INVALID_ARG
    assert call(ok_src, ok_dst, 0) == nb.NUNA_OK                               # empty: no launch, no context
    assert call(ok_src * 9, ok_dst * 9, 8) == nb.NUNA_ERR_TOO_MANY_RANKS
    assert call(ok_src, ok_dst, 8, dtype=nb.NUNA_F16) in (nb.NUNA_ERR_CUDA, nb.NUNA_OK)   # valid type; no device here
    assert call(ok_src, [A + 8192, A + 8192 + 16], 5, dtype=nb.NUNA_F32) == nb.NUNA_ERR_ALIAS   # 20 bytes each: overlap
    assert call(ok_src, [A + 8192, A + 8192 + 16], 5, dtype=nb.NUNA_BF16) in (nb.NUNA_ERR_CUDA, nb.NUNA_OK)  # 10 bytes: fine
    assert call(ok_src, ok_dst, 8, dtype=77) == nb.NUNA_ERR_UNSUPPORTED_DTYPE
    assert call(ok_src, ok_dst, 8, flags=3) == nb.NUNA_ERR_INVALID_ARG
    assert call(ok_src, ok_dst, 8, flags=1 << 15) == nb.NUNA_ERR_INVALID_ARG
    assert call(ok_src, ok_dst, 8, flags=nb.NUNA_CHAIN_PERSISTENT) == nb.NUNA_ERR_INVALID_ARG    # chain-only bit
    assert call(ok_src, [A + 8192, 0], 8) == nb.NUNA_ERR_INVALID_ARG
    assert call(ok_src, [A + 8192, A + 12288 + 2], 8) == nb.NUNA_ERR_ALIGNMENT
    assert call(ok_src, [A + 8192, A + 8192 + 16], 9) == nb.NUNA_ERR_ALIAS     # 18 bytes each: overlap
    assert call(ok_src, [A + 8192, A + 4096 + 2032], 2048) == nb.NUNA_ERR_ALIAS  # dst[1] inside src[1]
    assert call(ok_src, ok_dst, (1 << 40) + 1) == nb.NUNA_ERR_TOO_LARGE
    # shapes of the other collectives: allgather's destination is N times the shard
    ag = lambda *a, **k: nb.nuna_allgather(*a, stream=0, check=False, **k)
    assert ag(ok_src, [A + 8192, A + 8192 + 4096], 1024) in (nb.NUNA_ERR_CUDA, nb.NUNA_OK)  # valid; no device here
    assert ag(ok_src, [A + 8192, A + 8192 + 2048], 1024) == nb.NUNA_ERR_ALIAS  # needs 2*1024 elements = 4096 B each
    rs = lambda *a, **k: nb.nuna_reduce_scatter(*a, stream=0, check=False, **k)
    assert rs([A, A + 2048], ok_dst, 1024) in (nb.NUNA_ERR_CUDA, nb.NUNA_OK)   # sources may overlap each other
    assert rs(ok_src, [A + 2048, A + 12288], 1024) == nb.NUNA_ERR_ALIAS        # src[0] spans 2*1024 elements


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(nb, "_lib", None)
    monkeypatch.setattr(nb, "_LIB_PATH", "/nonexistent/libnuna.so")
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        nb.nuna_launch_count()

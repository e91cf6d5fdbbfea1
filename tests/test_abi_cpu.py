"""Host-side checks that need no GPU: the C-ABI library loads, exports every symbol the header declares,
and rejects bad arguments before launching anything."""
import ctypes as C
import os
import re

import pytest

import paper_2402_06262_b200 as R
from paper_2402_06262_b200.build import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    build()


def declared_functions():
    names = []
    for fn in sorted(os.listdir(os.path.join(ROOT, "include"))):
        text = open(os.path.join(ROOT, "include", fn)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names += re.findall(r"\b(roco_[a-z_0-9]+)\s*\(", text)
    return sorted(set(names))


def test_library_exports_every_declared_symbol():
    names = declared_functions()
    assert set(R.EXPORTS) <= set(names) and len(names) >= 8
    lib = C.CDLL(R.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in include/ but not exported"
    assert R.lib().roco_version() >= 100


def test_status_strings():
    assert R.status_string(0) == "ok"
    assert "workspace" in R.status_string(3)
    assert R.status_string(99) == "unknown status"


def fake_cache(**kw):
    """A struct with non-null, aligned but meaningless pointers: validation must fail before any use."""
    vals = dict(kv_dtype=R.ROCO_BF16, S=1, G=2, d=128, B=16)
    vals.update(kw)
    c = R.roco_cache(vals["kv_dtype"], vals["S"], vals["G"], vals["d"], vals["B"],
                     0x1000, 0x2000, 0x3000, 0x4000, 0x5000, 0x6000, 0x7000, 0x8000, 0x9000)
    for k in ("K", "V", "s", "q", "n", "pos", "live", "t_next", "status"):
        if k in kw:
            setattr(c, k, kw[k])
    return c


def decode(c, r=1, mode=R.ROCO_SCOPE_EXCLUDE_TOP_R, order=R.ROCO_EVICT_FIRST, q=0x10000, out=0x20000, ev=0x30000):
    return R.lib().roco_decode_step(C.byref(c), q, 0x11000, 0x12000, r, mode, order, 0.1, out, None, ev, None, None)


def test_decode_rejects_bad_arguments_on_the_host():
    L = R.lib()
    assert L.roco_decode_step(None, 1, 1, 1, 0, 0, 0, 0.1, 1, None, 1, None, None) == 1
    assert decode(fake_cache(K=None)) == 1
    assert decode(fake_cache(K=0x1008)) == 1                  # misaligned
    assert decode(fake_cache(d=96)) == 2                      # unsupported head dim
    assert decode(fake_cache(kv_dtype=7)) == 2
    assert decode(fake_cache(B=8193)) == 2
    assert decode(fake_cache(B=0)) == 1
    assert decode(fake_cache(), r=16) == 1                    # EXCLUDE_TOP_R needs r < B
    assert decode(fake_cache(), r=-1) == 1
    assert decode(fake_cache(), r=0, mode=R.ROCO_SCOPE_LOWEST_R) == 1
    assert decode(fake_cache(), r=17, mode=R.ROCO_SCOPE_LOWEST_R) == 1
    assert decode(fake_cache(), mode=5) == 1
    assert decode(fake_cache(), order=3) == 1
    assert decode(fake_cache(), q=None) == 1
    assert decode(fake_cache(), out=0x20004) == 1
    assert decode(fake_cache(), ev=None) == 1


def test_prefill_rejects_bad_arguments_on_the_host():
    L = R.lib()
    c = fake_cache()
    lens = (C.c_int32 * 1)(8)
    lp = C.cast(lens, C.c_void_p)
    need = L.roco_prefill_workspace_bytes(C.byref(c), 8)
    assert need > 0 and need % 256 == 0

    def call(Q=0x10000, lens_p=lp, Lmax=8, B=16, r=1, mode=0, cs=1, ws=0x100000, wsb=need):
        return L.roco_prefill(Q, 0x11000, 0x12000, lens_p, Lmax, B, r, mode, cs, 0.1, C.byref(c), None, None, None,
                              ws, wsb, None)
    assert call(Q=None) == 1
    assert call(B=8) == 1                                      # must equal cache->B
    assert call(r=17) == 1
    assert call(cs=0) == 2
    assert call(ws=None) == 3
    assert call(wsb=need - 1) == 3
    assert call(ws=0x100010) == 3                              # workspace must be 256-byte aligned
    assert call(Lmax=4) == 1                                   # lens > Lmax
    lens[0] = 0
    assert call() == 1
    lens[0] = 32
    assert call(Lmax=32, mode=R.ROCO_SCOPE_LOWEST_R, wsb=need) == 3      # LOWEST_R eviction needs the larger workspace
    assert L.roco_prefill_workspace_bytes_lowest_r(C.byref(c), 32) > L.roco_prefill_workspace_bytes(C.byref(c), 32)
    assert L.roco_prefill_workspace_bytes(None, 8) == 0
    assert L.roco_decode_host_staging_bytes(C.byref(c)) >= 4 * 2 * 128 * 2


def test_missing_library_fails_loudly(tmp_path, monkeypatch):
    from paper_2402_06262_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no fallback"):
        binding.lib()

"""The C-ABI library loads without a GPU, exports every declared symbol, and rejects bad arguments
before touching the device."""
import ctypes
import os
import re

import pytest

from paper_2306_15799_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "flurka.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(flurka_[a-z_0-9]+)\s*\(", text)))


def test_exports_every_declared_symbol(lib):
    names = _declared_symbols()
    assert "flurka_forward" in names and "flurka_forward_host" in names and len(names) >= 12
    for n in names:
        assert hasattr(lib, n), "libflurka.so does not export %s" % n
    assert sorted(binding.EXPORTS) == [n for n in names if n in binding.EXPORTS]
    assert set(binding.EXPORTS) <= set(names)
    assert lib.flurka_version() == 100


def test_strerror_is_static_text(lib):
    for code in range(-9, 1):
        s = lib.flurka_strerror(code)
        assert isinstance(s, bytes) and len(s) > 1
    assert b"NULL" in lib.flurka_strerror(-1)


def test_argument_checks_need_no_device(lib):
    buf = ctypes.create_string_buffer(1 << 16)
    base = (ctypes.addressof(buf) + 255) & ~255
    q, k, v, e, f, w, o = (base + 4096 * i for i in range(7))
    fwd = lib.flurka_forward
    ok = dict(variant=0, B=1, H=1, N=8, d=8, k=4, m=8)

    def call(Q=q, K=k, V=v, E=e, F=f, W=w, out=o, **kw):
        a = dict(ok); a.update(kw)
        return fwd(Q, K, V, E, F, W, a["variant"], a["B"], a["H"], a["N"], a["d"], a["k"], a["m"], out, None)

    assert call(Q=None) == -1 and call(out=None) == -1 and call(W=None) == -1
    assert call(W=None, variant=1) in (-7, 0)          # RNN needs no W; only the device is missing
    assert call(variant=7) == -2 and call(variant=0x800) == -2
    assert call(variant=0x200) in (-7, 0)              # [B,N,H,d] layout flag is valid
    assert call(N=0) == -3 and call(d=129) == -3 and call(k=0) == -3 and call(m=0) == -3 and call(k=5000) == -3
    assert call(B=70000) == -3
    assert call(Q=q + 2) == -4 and call(out=o + 8) == -4
    assert call(out=q) == -8 and call(out=e) == -8
    import torch
    if not torch.cuda.is_available():
        assert call() == -7                              # valid arguments, but no sm_100 device
    assert lib.flurka_workspace_bytes(0, 1, 2, 256, 32, 32, 64) > 2 * 2 * 32 * 32 * 4
    assert lib.flurka_workspace_bytes(9, 1, 2, 256, 32, 32, 64) == 0
    assert lib.flurka_set_workspace(ctypes.c_void_p(base + 8), 1024) == -4
    assert lib.flurka_set_workspace(None, 0) == 0
    prev = lib.flurka_set_path(1)
    assert lib.flurka_set_path(prev) == 1
    assert lib.flurka_debug_copy(0, ctypes.c_void_p(base), 16, None) == -5   # no forward has run yet


def test_binding_rejects_bad_tensors():
    import torch
    from paper_2306_15799_b200 import PERFORMER
    Q = torch.zeros(1, 1, 8, 8)
    E = torch.zeros(4, 8)
    W = torch.zeros(8, 8)
    with pytest.raises(ValueError):
        binding.flurka_forward(Q, Q, Q, E, E, W, PERFORMER)          # CPU tensors on the device entry
    with pytest.raises(ValueError):
        binding.flurka_forward_host(Q, Q, Q, torch.zeros(4, 9), E, W, PERFORMER, out=torch.zeros_like(Q))
    with pytest.raises(TypeError):
        binding.flurka_forward_host(Q.half(), Q.half(), Q.half(), E.half(), E.half(), W.half(), PERFORMER,
                                    out=torch.zeros_like(Q).half())

"""The C-ABI library builds, loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

from paper_1909_09010_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "gbmuf.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gbmuf_[a-z_]+)\s*\(", text)))


def test_library_builds_and_exports_the_header():
    path = build.build()
    assert os.path.exists(path)
    L = ctypes.CDLL(path)
    names = declared_symbols()
    assert "gbmuf_sync_round" in names and len(names) >= 10
    for n in names:
        assert hasattr(L, n), f"{n} is declared in gbmuf.h but not exported"
    assert sorted(binding.EXPORTS) == names, "binding and header disagree on the entry points"


def test_config_struct_layout_matches_header():
    # int32 K; int64 N, ld; int32 p, q; float eta, zeta; int32 mode, dtype; uint64 seed;
    # int32 device, comp_base; int64 elem_base  -> natural alignment
    C = binding.Config
    assert C.K.offset == 0 and C.N.offset == 8 and C.ld.offset == 16 and C.p.offset == 24
    assert C.q.offset == 28 and C.eta.offset == 32 and C.zeta.offset == 36 and C.mode.offset == 40
    assert C.theta_dtype.offset == 44 and C.seed.offset == 48 and C.device.offset == 56
    assert C.comp_base.offset == 60 and C.elem_base.offset == 64 and ctypes.sizeof(C) == 72


def test_argument_errors_need_no_gpu():
    """Validation happens before any CUDA call: these return INVALID_ARG on any machine."""
    L = binding.lib()
    h = ctypes.c_void_p()
    fake = ctypes.c_void_p(1 << 20)            # aligned, never dereferenced on these paths

    def create(**kw):
        base = dict(K=4, N=100, ld=128, p=1, q=1, eta=0.9, zeta=1.0, mode=0, theta_dtype=0, seed=0,
                    device=0, comp_base=0, elem_base=0)
        base.update(kw)
        cfg = binding.Config(**base)
        return L.gbmuf_create(ctypes.byref(cfg), fake, fake, fake, ctypes.byref(h))

    assert create(K=0) == binding.ERR_INVALID_ARG
    assert create(K=70000, p=1, q=1) == binding.ERR_UNSUPPORTED     # more than 256 workers
    assert create(N=0) == binding.ERR_INVALID_ARG
    assert create(ld=96) == binding.ERR_INVALID_ARG            # ld < N
    assert create(ld=130) == binding.ERR_INVALID_ARG           # not a multiple of 32
    assert create(q=3) == binding.ERR_INVALID_ARG              # q > min(2p, K-1)
    assert create(p=-1) == binding.ERR_INVALID_ARG
    assert create(mode=5) == binding.ERR_INVALID_ARG
    assert create(theta_dtype=2) == binding.ERR_INVALID_ARG
    assert create(comp_base=-1) == binding.ERR_INVALID_ARG
    assert create(eta=float("nan")) == binding.ERR_INVALID_ARG
    assert create(K=200, p=40, q=1) == binding.ERR_UNSUPPORTED  # more than 64 ring neighbours
    assert b"q exceeds" in L.gbmuf_last_error(None) or True
    assert create(q=3) == binding.ERR_INVALID_ARG and b"q exceeds" in L.gbmuf_last_error(None)
    cfg = binding.Config(4, 100, 128, 1, 1, 0.9, 1.0, 0, 0, 0, 0, 0, 0)
    assert L.gbmuf_create(ctypes.byref(cfg), None, fake, fake, ctypes.byref(h)) == binding.ERR_INVALID_ARG
    assert L.gbmuf_create(ctypes.byref(cfg), ctypes.c_void_p((1 << 20) + 4), fake, fake,
                          ctypes.byref(h)) == binding.ERR_INVALID_ARG
    assert L.gbmuf_create(None, fake, fake, fake, ctypes.byref(h)) == binding.ERR_INVALID_ARG
    assert h.value is None                                      # out untouched on every error
    assert L.gbmuf_destroy(None) == binding.GBMUF_OK
    assert L.gbmuf_sync_round(None, 0, None, None) == binding.ERR_INVALID_ARG

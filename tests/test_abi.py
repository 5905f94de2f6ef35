"""The C-ABI library loads, exports every symbol the header declares, and its host-side logic
(integer maps, descriptor validation) behaves as documented.  No GPU needed."""
import ctypes as C
import os
import re

import pytest
import torch

from oracle import kvcapsule_oracle as orc
from paper_2605_16439_b200 import binding as kvc
from paper_2605_16439_b200 import build as kvc_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    kvc_build.build()
    return kvc._lib()


def _declared_symbols():
    names = []
    inc = os.path.join(ROOT, "include")
    for f in sorted(os.listdir(inc)):
        if f.endswith(".h"):
            text = open(os.path.join(inc, f)).read()
            names += re.findall(r"KVC_API\s+[\w\s\*]+?\b(kvc_\w+)\s*\(", text)
    return names


def test_library_exports_every_declared_symbol(lib):
    names = _declared_symbols()
    assert {"kvc_compress", "kvc_decode_attend", "kvc_layer_create", "kvc_attend_full"} <= set(names)
    for name in names:
        assert hasattr(lib, name), f"{name} declared in include/ but not exported"


def test_retained_len_matches_oracle_bit_exactly(lib):
    for n in (1, 2, 7, 16, 256, 576, 1000, 1024, 4096):
        for r in (0, 1, 200, 333, 400, 600, 800, 950, 999):
            assert lib.kvc_retained_len(n, r) == orc.retained_len(n, r)
    assert lib.kvc_retained_len(0, 600) == -1 and lib.kvc_retained_len(16, 1000) == -1
    assert lib.kvc_retained_len(16, -1) == -1


def test_strerror_covers_all_codes(lib):
    seen = {lib.kvc_strerror(s).decode() for s in range(0, -9, -1)}
    assert len(seen) == 9 and "unknown status" not in seen
    assert lib.kvc_strerror(-99).decode() == "unknown status"


def _desc(**kw):
    d = kvc.kvc_layer_desc()
    d.layer, d.H_q, d.H_kv, d.d, d.n, d.ratio_permille, d.dtype = 0, 8, 2, 128, 16, 600, kvc.KVC_F32
    for k, v in kw.items():
        setattr(d, k, v)
    return d


def test_descriptor_validation_happens_on_the_host(lib):
    h = C.c_void_p()
    m = lib.kvc_retained_len(16, 600)
    good = (C.c_int32 * m)(*range(m))
    fake = C.c_void_p(256)         # never dereferenced: validation fails before any device work
    def create(**kw):
        d = _desc(**kw)
        return lib.kvc_layer_create(C.byref(d), C.byref(h))
    assert create(dtype=7, idx=good, theta=fake, U=fake, mu=fake) == -3
    assert create(d=64, idx=good, theta=fake, U=fake, mu=fake) == -2
    assert create(H_q=7, idx=good, theta=fake, U=fake, mu=fake) == -2
    assert create(H_q=64, H_kv=2, idx=good, theta=fake, U=fake, mu=fake) == -2      # G = 32 > 16
    assert create(ratio_permille=1000, idx=good, theta=fake, U=fake, mu=fake) == -2
    assert create(idx=good, theta=None, U=fake, mu=fake) == -4
    assert create(theta=fake, U=fake, mu=fake) == -4                                 # idx missing
    bad = (C.c_int32 * m)(*([0, 0] + list(range(2, m))))
    assert create(idx=bad, theta=fake, U=fake, mu=fake) == -8                        # not increasing
    bad2 = (C.c_int32 * m)(*(list(range(m - 1)) + [16]))
    assert create(idx=bad2, theta=fake, U=fake, mu=fake) == -8                       # out of range
    assert lib.kvc_layer_create(None, C.byref(h)) == -1
    assert lib.kvc_layer_destroy(None) == 0


def test_null_handle_calls_are_rejected(lib):
    assert lib.kvc_capsule_bytes(None, 1, 1) == 0
    assert lib.kvc_workspace_bytes(None, 1, 1, 1) == 0
    assert lib.kvc_compress(None, None, None, 1, 1, None, None) == -1
    assert lib.kvc_decode_attend(None, None, None, 1, 1, None, None, 0, 0, None, None, None) == -1
    assert lib.kvc_layer_m(None) == -1


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-GPU failure mode")
def test_product_path_fails_loudly_without_a_gpu(lib):
    with pytest.raises(kvc.KvcError) as e:
        kvc.Layer(8, 2, 128, 16, 0, torch.float32)
    assert e.value.status == -6

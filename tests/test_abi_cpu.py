"""Host-side checks of the C-ABI library that need no GPU: it loads, exports what include/mtpc.h declares,
validates configurations, and refuses to compute without a device (no CPU fallback)."""
import ctypes
import os
import re

import pytest

from paper_2511_11346_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "mtpc.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mtpc_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_functions()
    assert len(names) >= 11
    lib = B.lib()
    for name in names:
        assert hasattr(lib, name), name
    assert sorted(B.EXPORTS) == names


def cfg(**kw):
    base = dict(family=B.MTPC_CP, n=8, r=16, v=320, d=4096, io_dtype=B.MTPC_BF16, max_positions=8192,
                max_windows_per_pos=1, flags=0, v_valid=0)
    base.update(kw)
    return B.MtpcConfig(*[base[f] for f, _ in B.MtpcConfig._fields_])


def ws(c):
    out = ctypes.c_size_t(0)
    return B.lib().mtpc_workspace_bytes(ctypes.byref(c), ctypes.byref(out)), out.value


def test_workspace_bytes_for_the_named_configs():
    code, nbytes = ws(cfg())
    assert code == 0 and nbytes % 256 == 0
    # G [T, n, r] fp32 + log omega [T, r] fp32 + host-call staging of hidden dominate
    assert nbytes >= 8192 * 8 * 16 * 4 + 8192 * 16 * 4 + 8192 * 4096 * 2
    code, nb3 = ws(cfg(family=B.MTPC_BTREE, n=16, r=32, v=256, d=3072, max_positions=4096))
    assert code == 0 and nb3 >= 4096 * (1 + 14 * 32) * 32 * 4
    code, nb5 = ws(cfg(family=B.MTPC_HMM, r=32, flags=B.MTPC_FLAG_HMM_CONTEXTUAL))
    assert code == 0 and nb5 >= 8192 * (1 + 7 * 32) * 32 * 4   # contextual transitions: a table set per position
    code, nbp = ws(cfg(v=272, v_valid=268, d=3072))                   # byte-level Llama head: 268 symbols padded to 272
    assert code == 0 and nbp > 0
    code, nbv = ws(cfg(v=32768, r=2, n=2, max_positions=1024))        # large vocabularies plan (evaluation / training only)
    assert code == 0 and nbv > 0
    code, nb0 = ws(cfg(n=4, r=8, v=256, d=256, io_dtype=B.MTPC_F32, max_positions=256))
    assert code == 0 and nb0 >= 4 * 8 * 256 * 256 * 2       # bf16 copy of the fp32 weights lives in the workspace


@pytest.mark.parametrize("kw,code", [
    (dict(family=3), -2), (dict(n=0), -2), (dict(io_dtype=2), -2), (dict(max_positions=0), -2),
    (dict(v=272, v_valid=256), -2), (dict(v=272, v_valid=273), -2), (dict(v_valid=-3), -2),
    (dict(flags=1), -3), (dict(flags=2), -3), (dict(family=B.MTPC_BTREE, n=8, r=8, flags=1), -3), (dict(r=3), -3), (dict(r=256), -3), (dict(family=B.MTPC_HMM, r=64), -3),
    (dict(family=B.MTPC_BTREE, n=6, r=8), -3), (dict(family=B.MTPC_BTREE, n=1, r=8), -3), (dict(d=100), -3),
    (dict(v=100), -3), (dict(n=65), -3), (dict(max_windows_per_pos=65), -3),
])
def test_bad_configurations_are_refused(kw, code):
    got, _ = ws(cfg(**kw))
    assert got == code


def test_null_pointers_and_status_strings():
    lib = B.lib()
    out = ctypes.c_size_t(0)
    assert lib.mtpc_workspace_bytes(None, ctypes.byref(out)) == -1
    assert lib.mtpc_window_logprob(None, None, None, 0, None, None) == -1
    assert lib.mtpc_draft_sample(None, None, 0, 1, None, None, None, None) == -1
    assert lib.mtpc_destroy(None) == -1
    assert lib.mtpc_update_parameters(None, None, None, None, None) == -1
    assert lib.mtpc_lowrank_compose(1, 1, 16, 64, 2, None, None, None, None, None) == -1
    assert lib.mtpc_lowrank_backward(1, 1, 16, 64, 2, None, None, None, None, None, None, None) == -1
    fake = ctypes.c_void_p(256)           # never dereferenced: the argument checks come first
    assert lib.mtpc_lowrank_compose(1, 1, 16, 64, 0, fake, fake, fake, fake, None) == -2
    assert lib.mtpc_lowrank_compose(1, 1, 16, 64, 65, fake, fake, fake, fake, None) == -3
    assert lib.mtpc_lowrank_backward(1, 1, 2048, 64, 65, fake, fake, fake, fake, fake, fake, None) == -3
    seen = {B.status_string(c) for c in range(0, -8, -1)}
    assert len(seen) == 8 and "ok" in seen


def test_no_device_means_an_error_not_a_fallback():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    c = cfg(n=2, r=2, v=16, d=64, max_positions=4)
    handle = ctypes.c_void_p(0)
    fake = ctypes.c_void_p(256)           # never dereferenced: the device check comes first
    code = B.lib().mtpc_create_head(ctypes.byref(c), fake, fake, None, fake, 1 << 30, None, ctypes.byref(handle))
    assert code == -5 and not handle.value

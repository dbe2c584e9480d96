"""The C ABI library loads, exports every symbol the header declares, and validates arguments (no GPU needed)."""
import ctypes
import os
import re

import numpy as np
import pytest

import paper_2608_22704_b200 as wnw
from paper_2608_22704_b200 import build as wbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    """Every function declared in include/*.h (the decode path's interface and the test / measurement hooks)."""
    import glob
    names = set()
    for path in glob.glob(os.path.join(ROOT, "include", "*.h")):
        text = re.sub(r"/\*.*?\*/", "", open(path).read(), flags=re.S)
        names |= set(re.findall(r"\b(wnw_[a-z_]+)\s*\(", text))
    return sorted(names)


def test_library_builds_and_exports_every_declared_symbol():
    path = wbuild.build()
    lib = ctypes.CDLL(path)
    names = _declared()
    assert len(names) >= 18
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(wnw.exported_symbols()) == names      # the binding covers the whole header


def test_status_strings():
    assert wnw.status_string(0) == "ok"
    assert "argument" in wnw.status_string(wnw.WNW_ERR_INVALID_ARG)


@pytest.mark.parametrize("kw,status", [
    (dict(budget=0.0), wnw.WNW_ERR_INVALID_ARG),
    (dict(budget=1.5), wnw.WNW_ERR_INVALID_ARG),
    (dict(head_dim=96), wnw.WNW_ERR_UNSUPPORTED),
    (dict(chunk_tokens=0), wnw.WNW_ERR_INVALID_ARG),
    (dict(n_q_heads=7), wnw.WNW_ERR_INVALID_ARG),
    (dict(n_q_heads=4 * 32), wnw.WNW_ERR_UNSUPPORTED),
    (dict(topk=99), wnw.WNW_ERR_INVALID_ARG),
    (dict(roles=np.array([1, 1, 2, 2], np.uint8)), wnw.WNW_ERR_INVALID_ARG),     # tidal heads but no anchor
    (dict(roles=np.array([0, 1, 2, 7], np.uint8)), wnw.WNW_ERR_INVALID_ARG),
    (dict(max_batch=0), wnw.WNW_ERR_INVALID_ARG),
])
def test_create_rejects_bad_config_before_touching_the_device(kw, status):
    base = dict(n_layers=1, n_q_heads=8, n_kv_heads=4, head_dim=64, max_batch=1, max_audio_tokens=1024, max_text_tokens=64,
                chunk_tokens=32, budget=0.2, roles=np.array([0, 1, 1, 2], np.uint8))
    base.update(kw)
    with pytest.raises(wnw.WnwError) as e:
        wnw.wnw_create(**base)
    assert e.value.status == status


def test_null_handles_are_rejected():
    lib = wnw.lib()
    assert lib.wnw_destroy(None) == wnw.WNW_ERR_INVALID_ARG
    assert lib.wnw_sync(None) == wnw.WNW_ERR_INVALID_ARG
    assert lib.wnw_step_end(None, None) == wnw.WNW_ERR_INVALID_ARG
    assert lib.wnw_create(None, None) == wnw.WNW_ERR_INVALID_ARG

"""The C-ABI library without a GPU: it loads, exports every entry point the header declares, and its
host-side argument checks answer before anything touches a device."""
import ctypes as C
import os
import re

import pytest

from paper_2403_04643_b200 import qaq

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_names():
    text = open(os.path.join(ROOT, "include", "qaq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(qaq_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_entry_point_is_exported_and_bound():
    names = declared_names()
    assert {"qaq_select_bits", "qaq_quantize_append", "qaq_decode_attention", "qaq_outlier_thresholds"} <= set(names)
    L = qaq.lib()
    for n in names:
        assert hasattr(L, n), n
    assert set(names) == set(qaq.EXPORTED)


def test_status_strings():
    assert qaq.status_string(0) == "ok"
    assert "capacity" in qaq.status_string(3) and "workspace" in qaq.status_string(5)


def test_policy_from_hyper_matches_closed_form():
    import math
    p = qaq.qaq_policy_from_hyper(0.01, 0.05, 64.0, 512)
    sigK = math.sqrt(math.log(512**3 / 511 * 1e-4 + 1) / 64.0)
    assert p.cK == pytest.approx(2 * math.sqrt(3) * sigK, rel=1e-6)
    assert p.cV == pytest.approx(2 * math.sqrt(3) * 0.05 / math.sqrt(512), rel=1e-6)
    assert qaq.qaq_policy_from_hyper(0.01, 0.05, 64.0, 1).cK == 0.0


def test_bad_arguments_are_refused_on_the_host():
    L = qaq.lib()
    h = C.c_void_p()
    for bad in (qaq.make_config(1, 1, 48, 16), qaq.make_config(1, 1, 128, 16, bits_min=0),
                qaq.make_config(1, 1, 128, 16, bits_min=5, bits_max=3)):
        assert L.qaq_cache_create(C.byref(bad), C.byref(h)) == 2 and not h.value     # unsupported shape
    assert L.qaq_cache_create(C.byref(qaq.make_config(0, 1, 128, 16)), C.byref(h)) == 1
    assert L.qaq_cache_create(None, C.byref(h)) == 1
    n = C.c_size_t()
    assert L.qaq_decode_workspace_bytes(None, C.byref(n)) == 1
    assert L.qaq_cache_tokens(None) == -1
    cfg = qaq.make_config(1, 2, 128, 64)
    pol = qaq.Policy(0.1, 0.1)
    # null and misaligned pointers, bad strides: refused before any launch
    assert L.qaq_select_bits(C.byref(cfg), C.byref(pol), None, None, 0, 0, 128, 4, None, None, None, None, None, None) == 1
    assert L.qaq_outlier_thresholds(C.byref(cfg), None, None, 0, 0, 128, 4, None, None, 0, None) == 1
    assert L.qaq_thresholds_workspace_bytes(C.byref(cfg), C.byref(n)) == 0 and n.value > 0

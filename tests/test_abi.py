"""Host-side checks of the C-ABI library: it builds for sm_100a, loads, and
exports every symbol that include/gala.h declares (no compute calls: no GPU
is needed)."""
import ctypes
import os
import re

import pytest

from paper_1906_04585_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "gala.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gala_[a-z0-9_]+)\s*\(", text)))


def test_library_builds_and_exports_header_symbols():
    path = build.build()
    assert os.path.exists(path)
    lib = ctypes.CDLL(path)
    names = declared_symbols()
    assert len(names) >= 20
    for name in names:
        assert hasattr(lib, name), name
    assert sorted(binding.EXPORTS) == names


def test_binding_has_same_names():
    for name in declared_symbols():
        assert callable(getattr(binding, name)), name


def test_argument_validation_needs_no_gpu():
    L = binding.lib()
    h = ctypes.c_void_p()
    topo = binding.gala_topology(binding.GALA_TOPO_RING, 1)
    net = binding.gala_net_spec(binding.GALA_NET_MLP, 8, 64, 4, 0)
    hp = binding.default_hparams(16, 5)
    assert L.gala_create(0, ctypes.byref(topo), ctypes.byref(net), ctypes.byref(hp), ctypes.byref(h)) == binding.GALA_EINVAL
    bad = binding.gala_topology(7, 1)            # no such topology
    assert L.gala_create(4, ctypes.byref(bad), ctypes.byref(net), ctypes.byref(hp), ctypes.byref(h)) == binding.GALA_EINVAL
    hp2 = binding.default_hparams(16, 5, rms_eps=0.0)
    assert L.gala_create(4, ctypes.byref(topo), ctypes.byref(net), ctypes.byref(hp2), ctypes.byref(h)) == binding.GALA_EINVAL
    with pytest.raises(binding.GalaError):
        binding.gala_create(4, bad, net, hp)
    assert L.gala_destroy(None) == binding.GALA_EINVAL

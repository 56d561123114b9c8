"""The C ABI loads and exports every symbol include/tsdp.h declares; host-side argument checks."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2512_15773_b200 import binding, build, inputs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load_library()


def test_every_declared_symbol_is_exported(lib):
    hdr = open(os.path.join(ROOT, "include", "tsdp.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = set(re.findall(r"\b(tsdp_[a-z_]+)\s*\(", hdr))
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert getattr(lib, name) is not None


def test_struct_layouts_match_the_header():
    assert ctypes.sizeof(binding.NetT) == 20
    assert ctypes.sizeof(binding.ConfigT) == 2 * 20 + 16 * 4
    assert ctypes.sizeof(binding.AcceptT) == 16
    assert ctypes.sizeof(binding.StatsT) == 11 * 8 + 8 + 3 * 8 * 1024 + 5 * 8


def test_weight_counts_match_the_packer(lib):
    for name, wl in inputs.WORKLOADS.items():
        if name == "serving_xfmr":
            wl = dict(wl, base=dict(wl["base"], layers=2))
        if name == "robomimic_unet":
            wl = dict(wl, Do=16, base=dict(wl["base"], layers=2, d=128), draft=dict(wl["draft"], layers=1, d=128))
        if name == "vla_dit":                       # same architecture, sizes that a CPU test can afford
            wl = dict(wl, To=16, Do=32, base=dict(wl["base"], layers=2, d=256, heads=4),
                      draft=dict(wl["draft"], layers=1, d=128, heads=4))
        cfg = binding.make_config(wl["H"], wl["A"], wl["To"], wl["Do"], wl["base"], wl["draft"])
        for which, key in ((binding.BASE, "base"), (binding.DRAFT, "draft")):
            blob = binding.pack_weights(inputs.make_net(3, wl, key))
            assert lib.tsdp_weights_count(ctypes.byref(cfg), which) == blob.size
    g = binding.make_config(1, 1, 0, 0, dict(arch="gauss"), dict(arch="gauss"))
    assert lib.tsdp_weights_count(ctypes.byref(g), 0) == 2
    assert binding.pack_weights(inputs.make_gauss_params(0.7, 0.5)).tolist() == [np.float32(0.7), 0.5]


def test_bad_configs_are_rejected_without_touching_a_device(lib):
    h = ctypes.c_void_p()
    ok = dict(arch="xfmr", layers=1, d=128, heads=4)
    bad = [
        binding.make_config(16, 2, 2, 20, dict(arch="xfmr", layers=1, d=100, heads=4), ok),   # d % 128
        binding.make_config(16, 2, 2, 20, dict(arch="xfmr", layers=1, d=128, heads=3), ok),   # d % heads
        binding.make_config(16, 2, 2, 20, ok, ok, max_K=33),
        binding.make_config(16, 2, 2, 20, ok, ok, T=2000),
        binding.make_config(0, 2, 2, 20, ok, ok),
    ]
    for cfg in bad:
        assert lib.tsdp_init(ctypes.byref(cfg), ctypes.byref(h)) == 1
    cfg = binding.make_config(16, 2, 2, 20, ok, ok)
    cfg.base.arch = 9
    assert lib.tsdp_init(ctypes.byref(cfg), ctypes.byref(h)) == 7
    assert lib.tsdp_weights_count(ctypes.byref(cfg), 0) == 0
    assert lib.tsdp_init(None, ctypes.byref(h)) == 1
    assert lib.tsdp_strerror(5) == b"a bounded wait inside a kernel expired"


def test_no_cpu_fallback(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    cfg = binding.make_config(16, 2, 1, 20, dict(arch="mlp", layers=1, d=64), dict(arch="mlp", layers=1, d=64))
    with pytest.raises(binding.TsdpError) as e:
        binding.Sampler(cfg)
    assert e.value.status == 4

"""The shared library loads without a GPU, exports every symbol the header declares, and its
host-side logic (validation, arena sizing) answers without touching a device."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def ppu():
    from paper_2509_22418_b200 import build, ppu as mod
    build.build()
    return mod


def test_every_declared_symbol_is_exported(ppu):
    header = open(os.path.join(ROOT, "include", "ppu.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    names = set(re.findall(r"\b(ppu_[a-z0-9_]+)\s*\(", header))
    assert {"ppu_create", "ppu_local_step", "ppu_outer_sync", "ppu_loss"} <= names
    lib = ctypes.CDLL(ppu.LIB_PATH)
    for n in sorted(names):
        assert hasattr(lib, n), n


def test_struct_sizes_match_header(ppu):
    assert ctypes.sizeof(ppu.ModelCfg) == 7 * 4 + 9 * 4
    assert ctypes.sizeof(ppu.SubsetSpec) == 4 * 4 + 8 + 2 * 4 + 8
    assert ctypes.sizeof(ppu.Stats) == 6 * 8 + 4 * 8 + 8
    assert ctypes.sizeof(ppu.Profile) == 3 * 8 * 8 + 8


def test_query_bytes_and_validation_on_host(ppu):
    cfg = ppu.make_cfg(2, 64, 4, 256, 512, 4, 64)
    spec, _ = ppu.make_spec(4, n_slices=4)
    n = ppu.ppu_query_bytes(cfg, spec)
    params = 512 * 64 + 2 * (4 * 64 + 4 * 64 * 64 + 2 * 64 * 256) + 2 * 64
    assert n > params * 10          # fp32 params + momentum + bf16 copy at the very least
    # larger batch -> more activation memory; more replicas -> more state
    assert ppu.ppu_query_bytes(ppu.make_cfg(2, 64, 4, 256, 512, 8, 64), spec) > n
    spec8, _ = ppu.make_spec(8, n_slices=4)
    assert ppu.ppu_query_bytes(cfg, spec8) > n
    bad = [
        (ppu.make_cfg(2, 60, 4, 256, 512, 4, 64), spec),             # d_head 15
        (ppu.make_cfg(2, 64, 4, 252, 512, 4, 64), spec),             # d_ff not a multiple of 8
        (ppu.make_cfg(0, 64, 4, 256, 512, 4, 64), spec),
        (cfg, ppu.make_spec(6, n_slices=4)[0]),                      # K not a multiple of N
        (cfg, ppu.make_spec(4, n_slices=64)[0]),                     # slice narrower than 8
        (cfg, ppu.make_spec(4, ppu.SUBSET_FFN_LAYERS, layer_stride=5)[0]),
        (cfg, ppu.make_spec(1, ppu.SUBSET_EXPLICIT, ranges=[[[0, 12], [0, 8]]])[0]),
        (cfg, ppu.make_spec(1, ppu.SUBSET_EXPLICIT, ranges=[[[0, 512], [0, 8]]])[0]),
        (cfg, ppu.make_spec(4, n_slices=4, n_head_slices=3)[0]),     # 4 heads do not split in 3
        (cfg, ppu.make_spec(4, n_slices=4, train_non_mlp=2)[0]),
        (cfg, ppu.make_spec(4, n_slices=4, head_ranges=[[0, 1], [1, 2], [2, 5], [0, 4]])[0]),
    ]
    # training the never-sliced parameters and the projections costs state per replica
    assert ppu.ppu_query_bytes(cfg, ppu.make_spec(4, n_slices=4, train_non_mlp=1)[0]) > n
    assert ppu.ppu_query_bytes(cfg, ppu.make_spec(4, n_slices=4, n_head_slices=2)[0]) > n
    for c, s in bad:
        with pytest.raises(ppu.PpuError):
            ppu.ppu_query_bytes(c, s)


def test_compute_calls_fail_loudly_without_a_device(ppu):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    cfg = ppu.make_cfg(2, 64, 4, 256, 512, 4, 64)
    spec, keep = ppu.make_spec(4, n_slices=4)
    with pytest.raises(ppu.PpuError):
        ppu.Context(cfg, spec, keep)
    buf = ctypes.create_string_buffer(1 << 12)
    h = ctypes.c_void_p()
    addr = (ctypes.addressof(buf) + 255) & ~255
    rc = ppu.lib().ppu_create(ctypes.byref(cfg), ctypes.byref(spec), ctypes.c_void_p(addr),
                              ctypes.c_size_t(1 << 11), None, ctypes.byref(h))
    assert rc == -6 and not h.value

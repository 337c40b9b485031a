"""CPU-side checks of the C-ABI library: it loads, exports every symbol the
header declares, and validates its arguments before touching a device."""
import ctypes
import os
import re

import pytest

import paper_2410_14803_b200 as distrl
from paper_2410_14803_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    names = set()
    for f in os.listdir(os.path.join(ROOT, "include")):
        if f.endswith(".h"):
            text = open(os.path.join(ROOT, "include", f)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(distrl_[a-z_0-9]+)\s*\(", text))
    return names


def test_library_builds_and_exports_every_declared_symbol():
    path = build.build()
    lib = ctypes.CDLL(path)
    names = _declared_symbols()
    assert {"distrl_retrace_targets", "distrl_compute_priorities", "distrl_build_sampler", "distrl_sample",
            "distrl_update_priorities"} <= names
    for n in sorted(names):
        assert hasattr(lib, n), n


def test_version_and_error_strings():
    assert "sm_100a" in distrl.distrl_version()
    lib = binding._load()
    for code in range(0, -10, -1):
        assert lib.distrl_error_string(code)
    assert lib.distrl_error_string(-99) == b"unknown status"


def test_workspace_sizes_grow_and_are_aligned():
    prev = 0
    for n in (0, 1, 1000, 1 << 20, 1 << 24, 1 << 26):
        a, b = distrl.distrl_retrace_workspace_bytes(n), distrl.distrl_sampler_workspace_bytes(n)
        assert a % 256 == 0 and b % 256 == 0 and a >= 256 and b >= 256
        assert a + b >= prev
        prev = a + b
    # 2^24 masses: header, tree levels of 131072 + 4096 + 128 + 4 uint64 entries, one claim word per
    # mass, and the 65536-entry staging array of the refresh
    assert distrl.distrl_sampler_workspace_bytes(1 << 24) == \
        256 + 8 * (131072 + 4096 + 128) + 256 + 4 * (1 << 24) + 4 * 65536


def test_argument_validation_happens_before_any_device_work():
    lib = binding._load()
    b = binding.distrl_batch()
    assert lib.distrl_retrace_targets(None, 0.9, 0.9, None, None, None, None, None, None, 0, None) == binding.ERR_NULL
    assert lib.distrl_retrace_targets(ctypes.byref(b), 0.9, 0.9, None, None, None, None, None, None, 0, None) \
        == binding.ERR_SIZE                                      # struct_size not filled in
    b.struct_size = ctypes.sizeof(binding.distrl_batch)
    b.n_transitions = -1
    assert lib.distrl_retrace_targets(ctypes.byref(b), 0.9, 0.9, None, None, None, None, None, None, 0, None) \
        == binding.ERR_SIZE
    b.n_transitions = 8
    b.n_trajectories = 1
    assert lib.distrl_retrace_targets(ctypes.byref(b), 1.5, 0.9, None, None, None, None, None, None, 0, None) \
        == binding.ERR_PARAM
    assert lib.distrl_retrace_targets(ctypes.byref(b), 0.9, float("nan"), None, None, None, None, None, None, 0, None) \
        == binding.ERR_PARAM
    assert lib.distrl_retrace_targets(ctypes.byref(b), 0.9, 0.9, None, None, None, None, None, None, 0, None) \
        == binding.ERR_NULL
    b.n_transitions = 0                                          # empty batch: a no-op
    assert lib.distrl_retrace_targets(ctypes.byref(b), 0.9, 0.9, None, None, None, None, None, None, 0, None) == 0
    cfg = distrl.make_prio_cfg()
    assert lib.distrl_compute_priorities(0, None, None, None, None, ctypes.byref(cfg), None, None, None) == 0
    assert lib.distrl_compute_priorities(4, None, None, None, None, ctypes.byref(cfg), None, None, None) \
        == binding.ERR_NULL
    assert lib.distrl_compute_priorities(-4, None, None, None, None, ctypes.byref(cfg), None, None, None) \
        == binding.ERR_SIZE
    bad = distrl.make_prio_cfg(scale=0.0)
    assert lib.distrl_compute_priorities(4, None, None, None, None, ctypes.byref(bad), None, None, None) \
        == binding.ERR_PARAM
    assert lib.distrl_compute_priorities(4, None, None, None, None, None, None, None, None) == binding.ERR_NULL
    out = ctypes.c_void_p()
    assert lib.distrl_build_sampler(None, 10, None, 0, None, ctypes.byref(out)) == binding.ERR_NULL
    assert lib.distrl_sample(None, None, 1, 0.4, 1, None, None, None) == binding.ERR_NULL
    assert lib.distrl_update_priorities(None, None, 1, None, None, None, None, ctypes.byref(cfg), None, None) \
        == binding.ERR_NULL
    assert lib.distrl_destroy_sampler(None) == 0
    # circular buffer of trajectories
    rb = ctypes.c_void_p()
    assert lib.distrl_replay_create(0, 0, None, None, None, None, 1, None, 0, None, ctypes.byref(rb)) == binding.ERR_SIZE
    assert lib.distrl_replay_create(8, 9, None, None, None, None, 1, None, 0, None, ctypes.byref(rb)) == binding.ERR_SIZE
    assert lib.distrl_replay_create(8, 0, None, None, None, None, 1, None, 0, None, ctypes.byref(rb)) == binding.ERR_NULL
    assert lib.distrl_replay_create(8, 0, None, None, None, None, 1, None, 0, None, None) == binding.ERR_NULL
    assert lib.distrl_replay_ingest(None, None, 1, None, None, None, None, None, None) == binding.ERR_NULL
    assert lib.distrl_replay_head(None) == -1 and lib.distrl_replay_destroy(None) == 0
    assert distrl.distrl_replay_workspace_bytes(1 << 24) == 256 + 2 * (1 << 21) + 256 * ((513 * 8 + 255) // 256)
    assert lib.distrl_set_cooperative_launch(1) == 1
    # draws over several shards
    assert lib.distrl_route_draws(None, 1, None, 0, 0, None, None, None, None, None) == binding.ERR_PARAM
    assert lib.distrl_route_draws(None, 1, None, 65, 0, None, None, None, None, None) == binding.ERR_PARAM
    assert lib.distrl_route_draws(None, 1, None, 2, 2, None, None, None, None, None) == binding.ERR_PARAM
    assert lib.distrl_route_draws(None, 1, None, 2, 1, None, None, None, None, None) == binding.ERR_NULL
    assert lib.distrl_route_draws(None, 0, None, 2, 1, None, None, None, None, None) == binding.OK
    assert lib.distrl_finish_shard_draws(1, None, None, None, None, 2, 0, 0, 10, 0, 0.4, None, None, None) == binding.ERR_SIZE
    assert lib.distrl_finish_shard_draws(1, None, None, None, None, 2, 0, 20, 10, 0, 0.4, None, None, None) == binding.ERR_SIZE
    assert lib.distrl_finish_shard_draws(1, None, None, None, None, 2, 2, 5, 10, 0, 0.4, None, None, None) == binding.ERR_PARAM
    assert lib.distrl_finish_shard_draws(1, None, None, None, None, 2, 0, 5, 10, 0, 0.4, None, None, None) == binding.ERR_NULL
    assert lib.distrl_normalise_weights(None, 0, None) == binding.OK
    assert lib.distrl_normalise_weights(None, 3, None) == binding.ERR_NULL


def test_binding_refuses_host_tensors():
    import torch
    with pytest.raises(ValueError):
        binding._ptr(torch.zeros(4))

"""The C-ABI library loads on a machine without a GPU and exports what include/oda.h declares;
host-side validation rejects bad configurations.  No compute call is made here."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2609_20734_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "oda.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(oda_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    lib = binding.load_library()
    names = declared_symbols()
    assert {"oda_local_decode", "oda_recall_score", "oda_full_decode_gated", "oda_step"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in oda.h but missing from the library"
    assert set(names) == set(binding.EXPORTS)
    assert b"sm_100a" in lib.oda_version()


def base_cfg(**kw):
    L = kw.pop("L", 2)
    d = dict(num_layers=L, num_q_heads=8, num_kv_heads=2, head_dim=128, max_batch=4,
             max_blocks_per_seq=64, layer_window=[16] * L, layer_sinks=[4] * L, layer_gated=[1] * L,
             kv_layer_stride=64 * 2 * 16 * 128, kv_block_stride=2 * 16 * 128, kv_token_stride=128,
             kv_head_stride=16 * 128)
    d.update(kw)
    return binding.OdaConfig(**d)


def test_create_and_workspace_size_without_device_work():
    ctx = binding.OdaContext(base_cfg(), allocate_workspace=False)
    n = ctx.workspace_bytes()
    assert n > 0 and n % 256 == 0
    assert ctx.launch_count == 0
    bigger = binding.OdaContext(base_cfg(max_batch=64), allocate_workspace=False).workspace_bytes()
    assert bigger > n
    ctx.close()


@pytest.mark.parametrize("bad, status", [
    (dict(head_dim=96), 2), (dict(block_size=32), 2), (dict(num_q_heads=6, num_kv_heads=4), 1),
    (dict(num_q_heads=32, num_kv_heads=1), 2), (dict(max_batch=0), 1), (dict(max_batch=100000), 1),
    (dict(layer_window=[0, 16]), 1), (dict(layer_sinks=[-1, 0]), 1), (dict(kv_token_stride=100), 1),
    (dict(kv_token_stride=64), 1), (dict(out_dtype=3), 1), (dict(sm_scale=float("nan")), 1),
    (dict(variant=9), 1), (dict(num_layers=0, L=0), 1),
])
def test_create_rejects_bad_config(bad, status):
    with pytest.raises(binding.OdaError) as e:
        binding.OdaContext(base_cfg(**bad), allocate_workspace=False)
    assert e.value.status == status


def test_too_many_layer_classes_is_unsupported():
    L = 6
    with pytest.raises(binding.OdaError) as e:
        binding.OdaContext(base_cfg(L=L, layer_window=[8, 16, 24, 32, 40, 48]), allocate_workspace=False)
    assert e.value.status == 2


def test_calls_without_workspace_fail_cleanly():
    ctx = binding.OdaContext(base_cfg(), allocate_workspace=False)
    with pytest.raises(binding.OdaError) as e:
        ctx.local_decode(0, 2, 1, 256, 256, 256, 256, 256, 256, None, stream=0)
    assert e.value.status == 3
    with pytest.raises(binding.OdaError) as e:
        ctx.set_workspace(0, 1 << 30, stream=0)
    assert e.value.status == 3
    with pytest.raises(binding.OdaError) as e:
        ctx.set_workspace(128, 1 << 30, stream=0)   # misaligned
    assert e.value.status == 3
    with pytest.raises(binding.OdaError) as e:
        ctx.set_workspace(4096, 16, stream=0)       # too small
    assert e.value.status == 3
    assert binding.load_library().oda_status_string(3) == b"workspace missing or too small"


def test_host_only_calls_check_their_arguments():
    """An entry point that does no device work: a NULL context is refused, any budget is accepted."""
    lib = binding.load_library()
    assert lib.oda_set_cache_resident_bytes(None, 0) == 1
    ctx = binding.OdaContext(base_cfg(), allocate_workspace=False)
    ctx.set_cache_resident_bytes(64 << 20)
    ctx.set_cache_resident_bytes(0)
    ctx.close()


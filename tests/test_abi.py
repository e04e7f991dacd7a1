"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
header declares, sizes workspaces, and rejects bad arguments before launching anything."""
import ctypes
import os
import re

import pytest

from paper_2506_18145_b200 import binding as rb
from paper_2506_18145_b200 import build as rbuild
from paper_2506_18145_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    rbuild.build()
    return rb.lib()


def test_library_exports_every_declared_symbol(L):
    header = open(os.path.join(ROOT, "include", "rom.h")).read()
    declared = set(re.findall(r"ROM_API\s+(?:const\s+)?\w+\s*\*?\s*(rom_\w+)\s*\(", header))
    assert declared == set(rb.EXPORTS)
    for name in declared:
        assert hasattr(L, name), name


def test_status_strings(L):
    assert rb.status_string(0) == "ok"
    seen = {rb.status_string(c) for c in range(-6, 1)}
    assert len(seen) == 7 and "unknown status" not in seen
    assert rb.status_string(-99) == "unknown status"


def test_workspace_size_grows_with_the_problem_and_covers_named_taps(L):
    sizes = {}
    for name, s in synth.CONFIGS.items():
        cfg = rb.config_from_shape(s)
        n = rb.workspace_size(cfg)
        sizes[name] = n
        for tap in ("U", "delta_r", "Bm", "Cm", "Delta", "row_of_assign", "XZp", "Ygp", "pad_offsets"):
            off, nb = rb.workspace_find(cfg, tap)
            assert off % 256 == 0 and off + nb <= n
    assert sizes["tiny_fp32"] < sizes["small_bf16"] < sizes["long_ctx"] < sizes["short_seqs"]
    assert sizes["short_seqs"] < 8 << 30
    with pytest.raises(rb.RomError):
        rb.workspace_find(rb.config_from_shape(synth.CONFIGS["tiny_fp32"]), "nope")


def _cfg(**kw):
    base = dict(B=1, L=64, d_model=128, d_inner=256, d_state=16, d_conv=4, dt_rank=16, E=4, K=1, dtype="bf16")
    base.update(kw)
    return rb.make_config(**base)


@pytest.mark.parametrize("kw,code", [
    (dict(K=5), -1), (dict(K=0), -1), (dict(E=0), -1), (dict(E=65, K=1), -2), (dict(E=16, K=9), -2),
    (dict(d_model=100), -1), (dict(d_inner=200), -1), (dict(d_state=8), -2), (dict(d_conv=5), -2),
    (dict(d_conv=0), -1), (dict(dt_rank=0), -1), (dict(dt_rank=24), -2), (dict(B=0), -1), (dict(L=0), -1),
    (dict(gate_mode=2), -1), (dict(disc_mode=3), -1), (dict(flags=16), -1),
])
def test_layer_forward_rejects_bad_configs_on_the_host(L, kw, code):
    cfg = _cfg(**kw)
    w = rb.RomWeights(*([4096] * 11))
    rc = L.rom_layer_forward(ctypes.byref(cfg), ctypes.byref(w), 4096, 4096, None, None, None, 4096, 1 << 40, None)
    assert rc == code


def test_null_and_misaligned_pointers_and_small_workspace(L):
    cfg = _cfg()
    w = rb.RomWeights(*([4096] * 11))
    need = rb.workspace_size(cfg)
    f = lambda *a: L.rom_layer_forward(ctypes.byref(cfg), *a)
    assert f(None, 4096, 4096, None, None, None, 4096, need, None) == -1
    assert f(ctypes.byref(w), None, 4096, None, None, None, 4096, need, None) == -1
    assert f(ctypes.byref(w), 4096, None, None, None, None, 4096, need, None) == -1
    assert f(ctypes.byref(w), 4096, 4096, None, None, None, None, need, None) == -1
    assert f(ctypes.byref(w), 4100, 4096, None, None, None, 4096, need, None) == -1        # misaligned x
    assert f(ctypes.byref(w), 4096, 4096, None, None, None, 4096, need - 1, None) == -3    # workspace too small
    w2 = rb.RomWeights(*([4096] * 11)); w2.W_out = None
    assert f(ctypes.byref(w2), 4096, 4096, None, None, None, 4096, need, None) == -1
    # route / scan entry points
    assert L.rom_route(ctypes.byref(cfg), None, 4096, None, None, None, None, None, None, None, 4096, need, None) == -1
    assert L.rom_route(ctypes.byref(cfg), 4096, 4096, None, None, None, None, None, None, None, 4096, 16, None) == -3
    assert L.rom_scan(ctypes.byref(cfg), 4096, 4096, 4096, 4096, None, None, None, None, 4096, None, None, 0, None) == -1
    assert L.rom_workspace_size(None, None) == -1


def test_no_device_means_an_error_not_a_fallback(L):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    cfg = _cfg()
    w = rb.RomWeights(*([4096] * 11))
    need = rb.workspace_size(cfg)
    rc = L.rom_layer_forward(ctypes.byref(cfg), ctypes.byref(w), 4096, 4096, None, None, None, 4096, need, None)
    assert rc in (-4, -5)      # CUDA call failed / wrong device: never a silent CPU path

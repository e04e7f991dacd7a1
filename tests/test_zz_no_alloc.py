"""rom_route_noalloc, the routing entry point for hosts that may not allocate device memory (a
serving process with a fixed memory pool, an allocator locked after start-up): it keeps its scratch
in a fixed array inside the library instead of a caller workspace.  Checked here through the C ABI
against rom_route on the same inputs (every integer table bit for bit, gates exactly) and against the
CPU oracle's router and permutation tables, on two calls in a row that share the scratch (the second
one smaller, so stale contents of the first are still in the array when it runs).  Collected last on
purpose: a run that stops at the first failure has then already run every other test."""
import pytest
import torch

from paper_2506_18145_b200 import binding as rb
from paper_2506_18145_b200 import synth

from rom_testlib import check_route_exact, gpu_route

NAMES = ("idx", "gates", "counts", "offsets", "perm", "inv_perm")


def _route_noalloc(shape, p, gate_mode=0):
    cfg = rb.config_from_shape(shape, gate_mode)
    T, K, E = shape.T, shape.K, shape.E
    dev = "cuda"
    out = dict(idx=torch.empty((T, K), dtype=torch.int32, device=dev),
               gates=torch.empty((T, K), dtype=torch.float32, device=dev),
               counts=torch.empty((E,), dtype=torch.int32, device=dev),
               offsets=torch.empty((E + 1,), dtype=torch.int32, device=dev),
               perm=torch.empty((T * K,), dtype=torch.int32, device=dev),
               inv_perm=torch.empty((T * K,), dtype=torch.int32, device=dev))
    b_r = None if p["b_r"] is None else p["b_r"].to(dev)
    rb.rom_route_noalloc(cfg, p["x"].to(dev), p["W_r"].to(dev), b_r, out["idx"], out["gates"], out["counts"],
                         out["offsets"], out["perm"], out["inv_perm"])
    torch.cuda.synchronize()
    return {k: v.cpu().numpy() for k, v in out.items()}


@pytest.mark.gpu
def test_route_noalloc_matches_route_on_two_calls_in_a_row():
    first = synth.RomShape("na1", 3, 1111, 128, 64, 16, 4, 16, 8, 2, "bf16", 88000, router_bias_scale=1.0)
    second = synth.RomShape("na2", 1, 301, 256, 64, 16, 4, 16, 5, 1, "f32", 88100)
    for s in (first, second):
        p = synth.make_inputs(s, recipe="unit")
        want = gpu_route(s, p)                    # the existing entry point, caller-owned workspace
        got = _route_noalloc(s, p)
        for name in NAMES:
            assert (got[name] == want[name]).all(), f"{s.name}: {name} differs from rom_route"
        check_route_exact(got, s, p)              # and first-hand against the oracle


@pytest.mark.gpu
def test_route_noalloc_without_index_outputs_after_a_larger_call():
    """topk_idx = NULL and gates = NULL: the working copy of the indices then lives in the shared array, which
    still holds the indices of the larger call made just before."""
    big = synth.RomShape("na3", 2, 2000, 128, 64, 16, 4, 16, 8, 2, "bf16", 88300)
    _route_noalloc(big, synth.make_inputs(big, recipe="unit"))
    s = synth.RomShape("na4", 1, 257, 128, 64, 16, 4, 16, 6, 2, "bf16", 88400)
    p = synth.make_inputs(s, recipe="unit")
    want = gpu_route(s, p)
    cfg = rb.config_from_shape(s)
    T, K, E = s.T, s.K, s.E
    out = dict(counts=torch.empty((E,), dtype=torch.int32, device="cuda"), offsets=torch.empty((E + 1,), dtype=torch.int32, device="cuda"),
               perm=torch.empty((T * K,), dtype=torch.int32, device="cuda"), inv_perm=torch.empty((T * K,), dtype=torch.int32, device="cuda"))
    rb.rom_route_noalloc(cfg, p["x"].cuda(), p["W_r"].cuda(), None, None, None, out["counts"], out["offsets"], out["perm"], out["inv_perm"])
    torch.cuda.synchronize()
    for name, v in out.items():
        assert (v.cpu().numpy() == want[name]).all(), f"{name} differs from rom_route"


@pytest.mark.gpu
def test_route_noalloc_rejects_sizes_beyond_the_built_in_scratch():
    s = synth.RomShape("na_big", 1, 65537, 64, 64, 16, 4, 16, 4, 1, "bf16", 88200)
    cfg = rb.config_from_shape(s)
    x = torch.zeros((1, 8, 64), dtype=torch.bfloat16, device="cuda")     # never read: the call must not launch
    W = torch.zeros((4, 64), dtype=torch.bfloat16, device="cuda")
    rc = rb.rom_route_noalloc(cfg, x, W, None, None, None, None, None, None, None, check=False)
    assert rc == -7 and "built-in scratch" in rb.status_string(rc)
    s2 = s.replace(L=40000, K=4)                                         # tokens fit, assignments do not
    assert rb.rom_route_noalloc(rb.config_from_shape(s2), x, W, None, None, None, None, None, None, None, check=False) == -7


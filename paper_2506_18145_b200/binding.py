"""Thin ctypes binding of the C ABI declared in include/rom.h: argument marshalling only.

Every function takes torch tensors that already live where the ABI wants them (CUDA for data,
none on the host except sizes) and forwards raw pointers.  Nothing here computes anything; when
the compiled library is missing the import of `lib()` fails loudly -- there is no fallback.
"""
from __future__ import annotations

import ctypes
import os
from typing import Dict, Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "librom_b200.so")

ROM_F32, ROM_BF16 = 0, 1
ROM_FLAG_SIMT_GEMM = 1
ROM_FLAG_DEBUG_CHECKS = 2
ROM_FLAG_TEST_STALL = 4
ROM_FLAG_FUSED_SMALL = 8
ROM_OK = 0

EXPORTS = ("rom_workspace_size", "rom_route", "rom_scan", "rom_layer_forward", "rom_workspace_find",
           "rom_get_status", "rom_status_string", "rom_last_launch_count", "rom_layer_forward_profile",
           "rom_num_stages", "rom_stage_name", "rom_route_noalloc", "rom_route_balance",
           "rom_ffn_moe_workspace_size", "rom_ffn_moe_forward", "rom_layer_step", "rom_layer_forward_host",
           "rom_scan_workspace_size", "rom_debug_check", "rom_scan_backward_workspace_size", "rom_scan_backward",
           "rom_layer_backward_workspace_size", "rom_layer_backward", "rom_mamba2_workspace_size", "rom_mamba2_layer_forward")


class RomConfig(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("B", "L", "d_model", "d_inner", "d_state", "d_conv", "dt_rank", "E", "K", "dtype",
                 "gate_mode", "disc_mode", "flags", "small_proj_experts")]


class RomWeights(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in
                ("W_r", "b_r", "W_inz", "w_conv", "b_conv", "W_x", "W_dt", "b_dt", "A", "D", "W_out")]


class RomGrads(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in
                ("dW_r", "db_r", "dW_inz", "dw_conv", "db_conv", "dW_x", "dW_dt", "db_dt", "dA", "dD", "dW_out")]


class RomMamba2Weights(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in
                ("W_r", "b_r", "W_in", "w_conv", "b_conv", "dt_bias", "A", "D", "w_norm", "W_out")]


class RomError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} ({code})")


_lib = None


def lib() -> ctypes.CDLL:
    """Load librom_b200.so (built in-tree by paper_2506_18145_b200.build).  Raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2506_18145_b200.build` "
                              "(there is no CPU or PyTorch fallback)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32p, szp = ctypes.c_void_p, ctypes.c_void_p, ctypes.POINTER(ctypes.c_size_t)
        cfgp = ctypes.POINTER(RomConfig)
        L.rom_workspace_size.argtypes = [cfgp, szp]
        L.rom_scan_workspace_size.argtypes = [cfgp, szp]
        L.rom_debug_check.argtypes = [cfgp, vp, ctypes.c_size_t, vp]
        L.rom_scan_backward_workspace_size.argtypes = [cfgp, szp]
        L.rom_layer_backward_workspace_size.argtypes = [cfgp, szp]
        L.rom_mamba2_workspace_size.argtypes = [cfgp, ctypes.c_int32, szp]
        L.rom_mamba2_layer_forward.argtypes = [cfgp, ctypes.c_int32, ctypes.POINTER(RomMamba2Weights), vp, vp, i32p, vp, i32p, vp, ctypes.c_size_t, vp]
        L.rom_layer_backward.argtypes = [cfgp, ctypes.POINTER(RomWeights), vp, vp, vp, ctypes.POINTER(RomGrads), vp, ctypes.c_size_t, vp]
        L.rom_scan_backward.argtypes = [cfgp] + [vp] * 19 + [ctypes.c_size_t, vp]
        L.rom_route.argtypes = [cfgp, vp, vp, vp, i32p, vp, i32p, i32p, i32p, i32p, vp, ctypes.c_size_t, vp]
        L.rom_route_noalloc.argtypes = [cfgp, vp, vp, vp, i32p, vp, i32p, i32p, i32p, i32p, vp]
        L.rom_route_balance.argtypes = [cfgp, vp, vp, vp, ctypes.c_float, vp, vp, vp, vp, ctypes.c_size_t, vp]
        L.rom_ffn_moe_workspace_size.argtypes = [cfgp, ctypes.c_int32, szp]
        L.rom_ffn_moe_forward.argtypes = [cfgp, ctypes.c_int32, vp, vp, vp, i32p, vp, vp, vp, ctypes.c_size_t, vp]
        L.rom_scan.argtypes = [cfgp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, ctypes.c_size_t, vp]
        L.rom_layer_forward.argtypes = [cfgp, ctypes.POINTER(RomWeights), vp, vp, i32p, vp, i32p, vp, ctypes.c_size_t, vp]
        L.rom_layer_forward_host.argtypes = [cfgp, ctypes.POINTER(RomWeights), vp, vp, vp, vp, vp, ctypes.c_size_t, vp]
        L.rom_layer_step.argtypes = [cfgp, ctypes.POINTER(RomWeights), vp, vp, vp, vp, i32p, vp, vp, ctypes.c_size_t, vp]
        L.rom_workspace_find.argtypes = [cfgp, ctypes.c_char_p, szp, szp]
        L.rom_get_status.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_int32)]
        L.rom_status_string.argtypes = [ctypes.c_int]
        L.rom_status_string.restype = ctypes.c_char_p
        L.rom_last_launch_count.argtypes = []
        L.rom_layer_forward_profile.argtypes = [cfgp, ctypes.POINTER(RomWeights), vp, vp, vp, ctypes.c_size_t, vp,
                                                ctypes.POINTER(ctypes.c_float), ctypes.c_int]
        L.rom_num_stages.argtypes = []
        L.rom_stage_name.argtypes = [ctypes.c_int]
        L.rom_stage_name.restype = ctypes.c_char_p
        for name in EXPORTS:
            if name not in ("rom_status_string", "rom_stage_name"):
                getattr(L, name).restype = ctypes.c_int
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().rom_status_string(int(code)).decode()


def make_config(B, L, d_model, d_inner, d_state, d_conv, dt_rank, E, K, dtype, gate_mode=0, disc_mode=0, flags=0,
                small_proj_experts=0) -> RomConfig:
    dt = {"f32": ROM_F32, "bf16": ROM_BF16, torch.float32: ROM_F32, torch.bfloat16: ROM_BF16}[dtype]
    return RomConfig(B, L, d_model, d_inner, d_state, d_conv, dt_rank, E, K, dt, gate_mode, disc_mode, flags, small_proj_experts)


def config_from_shape(shape, gate_mode=0, disc_mode=0, flags=0, small_proj_experts=0) -> RomConfig:
    """shape: a synth.RomShape.  small_proj_experts: 0 = shared x Proj / dt Proj, shape.E = one per expert."""
    return make_config(shape.B, shape.L, shape.d_model, shape.d_inner, shape.d_state, shape.d_conv, shape.dt_rank,
                       shape.E, shape.K, shape.dtype, gate_mode, disc_mode, flags, small_proj_experts)


def _ptr(t: Optional[torch.Tensor], cuda: bool = True) -> Optional[int]:
    if t is None:
        return None
    if cuda and not t.is_cuda:
        raise ValueError("expected a CUDA tensor")
    if not t.is_contiguous():
        raise ValueError("expected a contiguous tensor")
    return t.data_ptr()


def _stream(stream: Optional[torch.cuda.Stream]) -> int:
    return (stream or torch.cuda.current_stream()).cuda_stream


def workspace_size(cfg: RomConfig) -> int:
    n = ctypes.c_size_t(0)
    rc = lib().rom_workspace_size(ctypes.byref(cfg), ctypes.byref(n))
    if rc != ROM_OK:
        raise RomError(rc, "rom_workspace_size")
    return int(n.value)


def scan_workspace_size(cfg: RomConfig) -> int:
    n = ctypes.c_size_t(0)
    rc = lib().rom_scan_workspace_size(ctypes.byref(cfg), ctypes.byref(n))
    if rc != ROM_OK:
        raise RomError(rc, "rom_scan_workspace_size", "rom_debug_check", "rom_scan_backward_workspace_size", "rom_scan_backward",
           "rom_layer_backward_workspace_size", "rom_layer_backward", "rom_mamba2_workspace_size", "rom_mamba2_layer_forward")
    return int(n.value)


def workspace_find(cfg: RomConfig, name: str):
    off, n = ctypes.c_size_t(0), ctypes.c_size_t(0)
    rc = lib().rom_workspace_find(ctypes.byref(cfg), name.encode(), ctypes.byref(off), ctypes.byref(n))
    if rc != ROM_OK:
        raise RomError(rc, "rom_workspace_find")
    return int(off.value), int(n.value)


def alloc_workspace(cfg: RomConfig, device="cuda") -> torch.Tensor:
    return torch.empty(workspace_size(cfg), dtype=torch.uint8, device=device)


def rom_route(cfg, x, W_r, b_r, topk_idx, gates, counts, offsets, perm, inv_perm, ws, stream=None, check=True) -> int:
    rc = lib().rom_route(ctypes.byref(cfg), _ptr(x), _ptr(W_r), _ptr(b_r), _ptr(topk_idx), _ptr(gates), _ptr(counts),
                         _ptr(offsets), _ptr(perm), _ptr(inv_perm), _ptr(ws), ws.numel() if ws is not None else 0, _stream(stream))
    if check and rc != ROM_OK:
        raise RomError(rc, "rom_route")
    return rc


def rom_route_noalloc(cfg, x, W_r, b_r, topk_idx, gates, counts, offsets, perm, inv_perm, stream=None, check=True) -> int:
    """rom_route without a workspace argument: the scratch is a fixed array inside the library
    (limits and sharing rules are stated beside the declaration in include/rom.h)."""
    rc = lib().rom_route_noalloc(ctypes.byref(cfg), _ptr(x), _ptr(W_r), _ptr(b_r), _ptr(topk_idx), _ptr(gates), _ptr(counts),
                                 _ptr(offsets), _ptr(perm), _ptr(inv_perm), _stream(stream))
    if check and rc != ROM_OK:
        raise RomError(rc, "rom_route_noalloc")
    return rc


def rom_route_balance(cfg, x, W_r, b_r, alpha, F, Pbar, loss, ws, stream=None, check=True) -> int:
    rc = lib().rom_route_balance(ctypes.byref(cfg), _ptr(x), _ptr(W_r), _ptr(b_r), ctypes.c_float(alpha), _ptr(F), _ptr(Pbar),
                                 _ptr(loss), _ptr(ws), ws.numel() if ws is not None else 0, _stream(stream))
    if check and rc != ROM_OK:
        raise RomError(rc, "rom_route_balance")
    return rc


def rom_scan(cfg, u, delta, A, Bm, Cm, D, z, h0, y, h_last, ws=None, stream=None, check=True) -> int:
    rc = lib().rom_scan(ctypes.byref(cfg), _ptr(u), _ptr(delta), _ptr(A), _ptr(Bm), _ptr(Cm), _ptr(D), _ptr(z), _ptr(h0),
                        _ptr(y), _ptr(h_last), _ptr(ws), ws.numel() if ws is not None else 0, _stream(stream))
    if check and rc != ROM_OK:
        raise RomError(rc, "rom_scan")
    return rc


def scan_backward_workspace_size(cfg: RomConfig) -> int:
    n = ctypes.c_size_t(0)
    rc = lib().rom_scan_backward_workspace_size(ctypes.byref(cfg), ctypes.byref(n))
    if rc != ROM_OK:
        raise RomError(rc, "rom_scan_backward_workspace_size")
    return int(n.value)


def rom_scan_backward(cfg, dy, u, delta, A, Bm, Cm, D, z, h0, dh_last, du, ddelta, dA, dBm, dCm, dD, dz, dh0, ws,
                      stream=None, check=True) -> int:
    rc = lib().rom_scan_backward(ctypes.byref(cfg), _ptr(dy), _ptr(u), _ptr(delta), _ptr(A), _ptr(Bm), _ptr(Cm), _ptr(D), _ptr(z),
                                 _ptr(h0), _ptr(dh_last), _ptr(du), _ptr(ddelta), _ptr(dA), _ptr(dBm), _ptr(dCm), _ptr(dD),
                                 _ptr(dz), _ptr(dh0), _ptr(ws), ws.numel() if ws is not None else 0, _stream(stream))
    if check and rc != ROM_OK:
        raise RomError(rc, "rom_scan_backward")
    return rc


def layer_backward_workspace_size(cfg: RomConfig) -> int:
    n = ctypes.c_size_t(0)
    rc = lib().rom_layer_backward_workspace_size(ctypes.byref(cfg), ctypes.byref(n))
    if rc != ROM_OK:
        raise RomError(rc, "rom_layer_backward_workspace_size")
    return int(n.value)


def make_grads(g: Dict[str, Optional[torch.Tensor]]) -> RomGrads:
    return RomGrads(*[_ptr(g.get(n)) for n, _ in RomGrads._fields_])


def rom_layer_backward(cfg, weights: RomWeights, x, dout, dx, grads: RomGrads, ws, stream=None, check=True) -> int:
    rc = lib().rom_layer_backward(ctypes.byref(cfg), ctypes.byref(weights), _ptr(x), _ptr(dout), _ptr(dx), ctypes.byref(grads), _ptr(ws),
                                  ws.numel() if ws is not None else 0, _stream(stream))
    if check and rc != ROM_OK:
        raise RomError(rc, "rom_layer_backward")
    return rc


def mamba2_workspace_size(cfg: RomConfig, headdim: int) -> int:
    n = ctypes.c_size_t(0)
    rc = lib().rom_mamba2_workspace_size(ctypes.byref(cfg), int(headdim), ctypes.byref(n))
    if rc != ROM_OK:
        raise RomError(rc, "rom_mamba2_workspace_size")
    return int(n.value)


def make_mamba2_weights(w: Dict[str, Optional[torch.Tensor]]) -> RomMamba2Weights:
    return RomMamba2Weights(*[_ptr(w.get(n)) for n, _ in RomMamba2Weights._fields_])


def rom_mamba2_layer_forward(cfg, headdim, weights: RomMamba2Weights, x, out, topk_idx_out, gates_out, counts_out, ws, stream=None, check=True) -> int:
    rc = lib().rom_mamba2_layer_forward(ctypes.byref(cfg), int(headdim), ctypes.byref(weights), _ptr(x), _ptr(out), _ptr(topk_idx_out),
                                        _ptr(gates_out), _ptr(counts_out), _ptr(ws), ws.numel() if ws is not None else 0, _stream(stream))
    if check and rc != ROM_OK:
        raise RomError(rc, "rom_mamba2_layer_forward")
    return rc


def make_weights(w: Dict[str, Optional[torch.Tensor]]) -> RomWeights:
    return RomWeights(*[_ptr(w.get(n)) for n, _ in RomWeights._fields_])


def rom_layer_forward(cfg, weights: RomWeights, x, out, topk_idx_out, gates_out, counts_out, ws, stream=None, check=True) -> int:
    rc = lib().rom_layer_forward(ctypes.byref(cfg), ctypes.byref(weights), _ptr(x), _ptr(out), _ptr(topk_idx_out),
                                 _ptr(gates_out), _ptr(counts_out), _ptr(ws), ws.numel() if ws is not None else 0, _stream(stream))
    if check and rc != ROM_OK:
        raise RomError(rc, "rom_layer_forward")
    return rc


def ffn_moe_workspace_size(cfg: RomConfig, d_ff: int) -> int:
    n = ctypes.c_size_t(0)
    rc = lib().rom_ffn_moe_workspace_size(ctypes.byref(cfg), int(d_ff), ctypes.byref(n))
    if rc != ROM_OK:
        raise RomError(rc, "rom_ffn_moe_workspace_size")
    return int(n.value)


def rom_ffn_moe_forward(cfg, d_ff, W_gu, W_down, x, topk_idx, gates, out, ws, stream=None, check=True) -> int:
    rc = lib().rom_ffn_moe_forward(ctypes.byref(cfg), int(d_ff), _ptr(W_gu), _ptr(W_down), _ptr(x), _ptr(topk_idx), _ptr(gates),
                                   _ptr(out), _ptr(ws), ws.numel() if ws is not None else 0, _stream(stream))
    if check and rc != ROM_OK:
        raise RomError(rc, "rom_ffn_moe_forward")
    return rc


def rom_layer_forward_host(cfg, weights: RomWeights, x_host, out_host, x_dev, out_dev, ws, stream=None, check=True) -> int:
    """x_host / out_host: CPU tensors (pinned for asynchronous copies); x_dev / out_dev: CUDA staging tensors."""
    rc = lib().rom_layer_forward_host(ctypes.byref(cfg), ctypes.byref(weights), _ptr(x_host, cuda=False), _ptr(out_host, cuda=False),
                                      _ptr(x_dev), _ptr(out_dev), _ptr(ws), ws.numel() if ws is not None else 0, _stream(stream))
    if check and rc != ROM_OK:
        raise RomError(rc, "rom_layer_forward_host")
    return rc


def rom_layer_step(cfg, weights: RomWeights, x, conv_state, ssm_state, out, topk_idx_out, gates_out, ws, stream=None, check=True) -> int:
    rc = lib().rom_layer_step(ctypes.byref(cfg), ctypes.byref(weights), _ptr(x), _ptr(conv_state), _ptr(ssm_state), _ptr(out),
                              _ptr(topk_idx_out), _ptr(gates_out), _ptr(ws), ws.numel() if ws is not None else 0, _stream(stream))
    if check and rc != ROM_OK:
        raise RomError(rc, "rom_layer_step")
    return rc


def rom_debug_check(cfg, ws, stream=None, check=True) -> int:
    rc = lib().rom_debug_check(ctypes.byref(cfg), _ptr(ws), ws.numel(), _stream(stream))
    if check and rc != ROM_OK:
        raise RomError(rc, "rom_debug_check")
    return rc


def rom_get_status(ws, stream=None) -> int:
    code = ctypes.c_int32(0)
    rc = lib().rom_get_status(_ptr(ws), _stream(stream), ctypes.byref(code))
    if rc != ROM_OK:
        raise RomError(rc, "rom_get_status")
    return int(code.value)


def last_launch_count() -> int:
    return int(lib().rom_last_launch_count())


def stage_names():
    L = lib()
    return [L.rom_stage_name(i).decode() for i in range(L.rom_num_stages())]


def rom_layer_forward_profile(cfg, weights: RomWeights, x, out, ws, stream=None):
    """Returns {stage name: milliseconds} of one forward (synchronises the stream)."""
    L = lib()
    n = L.rom_num_stages()
    ms = (ctypes.c_float * n)()
    rc = L.rom_layer_forward_profile(ctypes.byref(cfg), ctypes.byref(weights), _ptr(x), _ptr(out), _ptr(ws), ws.numel(),
                                     _stream(stream), ms, n)
    if rc != ROM_OK:
        raise RomError(rc, "rom_layer_forward_profile")
    return dict(zip(stage_names(), [float(v) for v in ms]))

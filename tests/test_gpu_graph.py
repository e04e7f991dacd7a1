"""The entry points allocate nothing and never synchronise: a call can be captured in a CUDA graph and replayed.

The replayed result must equal the directly launched one bit for bit (same kernels, same launch shapes, same buffers)."""
import pytest
import torch

from paper_2506_18145_b200 import binding as rb
from paper_2506_18145_b200 import synth

pytestmark = pytest.mark.gpu


def _capture(call):
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        call()                       # warm-up outside the capture: lazy one-time host initialisation happens here
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        call()
    return g


@pytest.mark.parametrize("name", ["tiny_fp32", "small_bf16"])
def test_layer_forward_replays_from_a_cuda_graph(name):
    s = synth.CONFIGS[name]
    p = synth.make_inputs(s, recipe="unit", with_D=False)
    d = {k: (None if v is None else v.cuda()) for k, v in p.items()}
    cfg = rb.config_from_shape(s)
    weights = rb.make_weights(d)
    ws = rb.alloc_workspace(cfg, "cuda")
    out = torch.empty_like(d["x"])
    call = lambda: rb.rom_layer_forward(cfg, weights, d["x"], out, None, None, None, ws)
    call()
    torch.cuda.synchronize()
    assert rb.rom_get_status(ws) == 0
    ref = out.clone()
    g = _capture(call)
    for _ in range(2):
        out.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert rb.rom_get_status(ws) == 0
        assert torch.equal(out, ref)


def test_layer_step_replays_from_a_cuda_graph():
    """Three generation steps: replaying the captured step advances the carried states exactly as three direct calls do."""
    s = synth.CONFIGS["small_bf16"].replace(B=8, L=1)
    p = synth.make_inputs(s, recipe="unit", with_D=False)
    d = {k: (None if v is None else v.cuda()) for k, v in p.items()}
    cfg = rb.config_from_shape(s)
    weights = rb.make_weights(d)
    ws = rb.alloc_workspace(cfg, "cuda")
    x_t = d["x"][:, 0].contiguous()
    out = torch.empty_like(x_t)

    def fresh():
        return (torch.zeros((s.B, s.d_conv - 1, s.d_inner), dtype=torch.float32, device="cuda"),
                torch.zeros((s.B, s.d_inner, s.d_state), dtype=torch.float32, device="cuda"))

    conv_state, ssm_state = fresh()
    call = lambda: rb.rom_layer_step(cfg, weights, x_t, conv_state, ssm_state, out, None, None, ws)
    outs = []
    for _ in range(3):
        call()
        torch.cuda.synchronize()
        outs.append(out.clone())
    ref_conv, ref_ssm = conv_state.clone(), ssm_state.clone()
    g = _capture(call)                 # (the warm-up and the capture itself do not run the step on the real states:
    z0, z1 = fresh()                   #  reset them before replaying)
    conv_state.copy_(z0); ssm_state.copy_(z1)
    for i in range(3):
        g.replay()
        torch.cuda.synchronize()
        assert rb.rom_get_status(ws) == 0
        assert torch.equal(out, outs[i])
    assert torch.equal(conv_state, ref_conv) and torch.equal(ssm_state, ref_ssm)

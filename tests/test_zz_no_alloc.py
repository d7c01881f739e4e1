"""moe_router_wgrad_static is the one entry point for callers that may not allocate device memory (a plug-in whose
host application owns all device memory, a loop that cannot absorb cudaMalloc's device-wide synchronisation): its
scratch is a fixed array inside the library.  This file is named so that pytest collects it last; a run that stops
at the first failure has then already run every other test.

The check: its dW_r equals the dW_r that moe_backward produces from the same x and the same router-logit gradient
dl (read back from the workspace), on two calls in a row with different shapes, so that whatever the first call
left in the shared scratch cannot leak into the second."""
import ctypes as C

import pytest
import torch

from paper_2608_00916_b200 import binding, synth
from gpu_util import Run, rel_fro

pytestmark = pytest.mark.gpu


def backward_reference(shape, seed):
    inp = synth.make_inputs(shape, seed, x_std=1.0)
    r = Run(inp, shape.k)
    r.forward()
    bw = r.backward(0.05)
    dl = r.layer.buffer("dl", torch.float32).view(shape.T, shape.E).clone()
    return r.dev["x"], dl, bw["dW_r"].clone()


def test_static_scratch_entry_matches_backward_twice_in_a_row():
    # first call: a larger problem fills the scratch; second call: a smaller one with a different E must not see it
    for shape, seed in ((synth.MoEShape(1500, 512, 64, 4, 128), 41), (synth.MoEShape(333, 192, 24, 3, 64), 42)):
        x, dl, want = backward_reference(shape, seed)
        got = binding.router_wgrad_static(x, dl)
        torch.cuda.synchronize()
        assert rel_fro(got.cpu().numpy(), want.cpu().numpy()) <= 1e-2
        # fp64 host contraction of the same operands: the static path is plain fp32 arithmetic
        ref = x.double().cpu().numpy().T @ dl.double().cpu().numpy()
        assert rel_fro(got.cpu().numpy(), ref) <= 1e-5
    # same inputs again, output buffer reused: bitwise the same result
    again = binding.router_wgrad_static(x, dl, dW_r=torch.empty_like(got))
    torch.cuda.synchronize()
    assert torch.equal(again, got)


def test_static_scratch_entry_at_its_size_limit_and_smallest_expert_count():
    """d * E exactly at the limit with the widest register tile (E = 256), then the narrowest (E = 8), back to back on
    the shared scratch; reference: the same contraction in float64 on the host."""
    assert 1024 * 256 == binding.STATIC_MAX_DE
    g = torch.Generator(device="cpu").manual_seed(7)
    for T, d, E in ((700, 1024, 256), (257, 1024, 8)):
        x = torch.randn(T, d, generator=g).to(torch.bfloat16).cuda()
        dl = (0.01 * torch.randn(T, E, generator=g)).cuda()
        got = binding.router_wgrad_static(x, dl)
        torch.cuda.synchronize()
        ref = x.double().cpu().numpy().T @ dl.double().cpu().numpy()
        assert rel_fro(got.cpu().numpy(), ref) <= 1e-5, (T, d, E)


def test_static_scratch_entry_refuses_shapes_beyond_its_scratch():
    lib = binding.load_library()
    d, E = 4096, 128  # d * E = 524288 > MOE_STATIC_MAX_DE
    assert d * E > binding.STATIC_MAX_DE
    x = torch.zeros(8, d, dtype=torch.bfloat16, device="cuda")
    dl = torch.zeros(8, E, dtype=torch.float32, device="cuda")
    out = torch.full((d, E), 7.0, dtype=torch.float32, device="cuda")
    rc = lib.moe_router_wgrad_static(8, d, E, C.c_void_p(x.data_ptr()), C.c_void_p(dl.data_ptr()),
                                     C.c_void_p(out.data_ptr()), None)
    assert rc == -2 and b"unsupported" in lib.moe_status_string(rc)
    torch.cuda.synchronize()
    assert bool((out == 7.0).all())  # nothing was launched
    with pytest.raises(binding.MoEError):
        binding.router_wgrad_static(x, dl)
    # T = 0 is legal and yields zeros
    z = binding.router_wgrad_static(torch.zeros(0, 256, dtype=torch.bfloat16, device="cuda"),
                                    torch.zeros(0, 16, dtype=torch.float32, device="cuda"))
    torch.cuda.synchronize()
    assert not z.cpu().numpy().any()

"""The C-ABI library loads and exports every symbol include/moe.h declares; host-side argument checks and the
workspace arithmetic run without a GPU (no kernel is launched here)."""
import ctypes as C
import os
import re

import pytest

from paper_2608_00916_b200 import binding
from paper_2608_00916_b200 import build as pbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    pbuild.build()
    return binding.load_library()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "moe.h")).read()
    return re.findall(r"MOE_API\s+[\w\s\*]+?\b(moe_\w+)\s*\(", text)


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert len(names) >= 12
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(names) == sorted(binding.EXPORTS)


def test_create_validates_arguments(lib):
    h = C.c_void_p()
    for bad in [(100, 8, 128, 2), (128, 0, 128, 1), (128, 300, 128, 2), (128, 8, 128, 9), (128, 8, 100, 2),
                (128, 64, 128, 33)]:
        cfg = binding.MoEConfig(*bad, 0)
        assert lib.moe_create(C.byref(cfg), C.byref(h)) == -1, bad
    cfg = binding.MoEConfig(2048, 128, 768, 8, 0)
    assert lib.moe_create(C.byref(cfg), C.byref(h)) == 0
    lib.moe_destroy(h)
    assert lib.moe_status_string(0) == b"ok" and b"workspace" in lib.moe_status_string(-3)


def test_workspace_arithmetic(lib):
    layer = binding.MoELayer(2048, 128, 768, 8)
    sizes = [layer.workspace_bytes(T) for T in (0, 1, 1000, 16384, 65536)]
    assert all(a < b for a, b in zip(sizes, sizes[1:]))
    assert lib.moe_workspace_bytes(None, 5) == 0 and layer.workspace_bytes(-1) == 0
    T = 16384
    rows_max = ((T * 8 + 127) // 128 + 128) * 128
    off, n = layer.find(T, "xp")
    assert n == rows_max * 2048 * 2 and off % 256 == 0
    off2, n2 = layer.find(T, "act")
    assert n2 == rows_max * 768 * 2 and off2 >= off + n
    assert layer.workspace_bytes(T) < 3 * 2**30  # saved activations of the Qwen shape fit in a few GB
    with pytest.raises(binding.MoEError):
        layer.find(T, "nonsense")
    # regions do not overlap
    spans = sorted(layer.find(T, nm) for nm in ("counts", "offsets", "pad_offsets", "logits", "idx", "gates", "inv",
                                                 "row_gate", "xp", "hg", "hu", "act", "o", "dhg", "dhu", "dxp", "dg",
                                                 "dl"))
    for (o1, n1), (o2, _) in zip(spans, spans[1:]):
        assert o1 + n1 <= o2


def test_forward_rejects_bad_arguments_before_launch(lib):
    layer = binding.MoELayer(128, 8, 128, 2)
    vp = C.c_void_p
    fake = vp(4096)  # aligned non-null pointer; never dereferenced because the checks fail first
    # T < 0
    args = [layer.h, -1] + [fake] * 14 + [fake, 1 << 30, None]
    assert lib.moe_forward(*args) == -1
    # workspace too small
    args = [layer.h, 64] + [fake] * 14 + [fake, 16, None]
    assert lib.moe_forward(*args) == -3
    # misaligned x
    args = [layer.h, 64, vp(4098)] + [fake] * 13 + [fake, 1 << 30, None]
    assert lib.moe_forward(*args) == -1
    # missing weights
    args = [layer.h, 64, fake, fake, None, None, None, fake, fake] + [fake] * 7 + [fake, 1 << 30, None]
    assert lib.moe_forward(*args) == -1


def test_other_entry_points_reject_bad_arguments_before_launch(lib):
    """Argument errors of backward, the LoRA variant, the host-step calls and the static-scratch entry are reported as
    codes without touching a device (the pointers are fakes that are never dereferenced)."""
    layer = binding.MoELayer(128, 8, 128, 2)
    vp = C.c_void_p
    fake = vp(4096)
    big = 1 << 40
    # backward: T < 0, missing dW buffers, small workspace
    assert lib.moe_backward(layer.h, -1, fake, C.c_float(0), *([fake] * 11), fake, big, None) == -1
    assert lib.moe_backward(layer.h, 8, fake, C.c_float(0), fake, fake, fake, fake, fake, fake, fake, None, None, fake,
                            fake, fake, big, None) == -1
    assert lib.moe_backward(layer.h, 8, fake, C.c_float(0), *([fake] * 11), fake, 64, None) == -3
    assert lib.moe_backward_accumulate(layer.h, 8, fake, C.c_float(0), fake, fake, fake, fake, fake, fake, fake, None,
                                       None, fake, fake, fake, big, None) == -1
    # LoRA: rank must be a multiple of 8 in [8, 64]; adapters must be present
    for bad_rank in (0, 4, 12, 72):
        assert lib.moe_lora_forward(layer.h, 8, bad_rank, C.c_float(1), *([fake] * 16), fake, big, None) == -1
    args = [fake] * 16
    args[6] = None  # A1 missing
    assert lib.moe_lora_forward(layer.h, 8, 16, C.c_float(1), *args, fake, big, None) == -1
    assert lib.moe_lora_forward(layer.h, 8, 16, C.c_float(1), *([fake] * 16), fake, 64, None) == -3
    assert layer.lib.moe_lora_workspace_bytes(layer.h, 64) > layer.workspace_bytes(64) > layer.inference_workspace_bytes(64)
    # host steps: bad slot, missing buffers, small device buffer
    assert lib.moe_step_host_begin(layer.h, 2, 8, fake, fake, C.c_float(0), fake, fake, fake, fake, big, None) == -1
    assert lib.moe_step_host_begin(layer.h, 0, 8, None, fake, C.c_float(0), fake, fake, fake, fake, big, None) == -1
    assert lib.moe_step_host_begin(layer.h, 0, 8, fake, fake, C.c_float(0), fake, fake, fake, fake, 64, None) == -3
    assert lib.moe_step_host_end(layer.h, 0) == -1  # nothing was begun
    assert lib.moe_step_host(layer.h, 8, 0, None, *([fake] * 5), C.c_float(0), *([fake] * 7), fake, big, None) == -1
    # static-scratch entry: shape limits
    assert lib.moe_router_wgrad_static(8, 100, 8, fake, fake, fake, None) == -1      # d not a multiple of 64
    assert lib.moe_router_wgrad_static(8, 128, 300, fake, fake, fake, None) == -1    # E > 256
    assert lib.moe_router_wgrad_static(8, 4096, 128, fake, fake, fake, None) == -2   # beyond the built-in scratch
    assert lib.moe_selftest_timeout(None, fake, None) == -1


def test_context_binds_to_a_device_only_when_work_is_launched(lib):
    """The per-device state of a context (SM count, tensor-map encoder, the kernels' shared-memory attributes) is
    set up by the first call that launches work and belongs to the device current then.  Without a device the call
    fails with a CUDA error and the context stays unbound; argument errors never bind it."""
    import torch
    layer = binding.MoELayer(128, 8, 128, 2)
    assert lib.moe_ctx_device(layer.h) == -1 and lib.moe_ctx_device(None) == -1
    vp = C.c_void_p
    fake = vp(4096)
    assert lib.moe_forward(layer.h, -1, *([fake] * 14), fake, 1 << 30, None) == -1
    assert lib.moe_ctx_device(layer.h) == -1
    if not torch.cuda.is_available():
        # valid arguments, but no device to bind to: reported as a CUDA failure before any pointer is touched
        assert lib.moe_forward(layer.h, 8, *([fake] * 14), fake, 1 << 30, None) == -4
        assert lib.moe_ctx_device(layer.h) == -1
    assert lib.moe_kernel_launches() >= 0

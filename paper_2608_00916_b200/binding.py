"""ctypes binding of the C ABI in include/moe.h.  Argument marshalling only: every step of the layer runs in
the CUDA library.  torch supplies device memory and the current stream; there is no fallback path - if the
shared library is missing or the device is not an sm_100a GPU, calls raise."""
from __future__ import annotations

import ctypes as C
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmoe_b200.so")
NUM_STAGES = 16
FLAG_CTA_PAIR_TILES = 1    # MOE_FLAG_CTA_PAIR_TILES of include/moe.h
FLAG_SINGLE_CTA_TILES = 2  # MOE_FLAG_SINGLE_CTA_TILES
FLAG_NO_SIDE_STREAM = 8    # MOE_FLAG_NO_SIDE_STREAM
FLAG_HYBRID_TILES = 16     # MOE_FLAG_HYBRID_TILES
FLAG_ROUTER_FP32 = 32      # MOE_FLAG_ROUTER_FP32
FLAG_DEBUG_CHECKS = 64     # MOE_FLAG_DEBUG_CHECKS
STAGE_NAMES = ["router", "permute", "gemm_gateup_swiglu", "gemm_down", "combine", "combine_bwd",
               "dgrad_down_swiglu_bwd", "wgrad_down", "dgrad_gateup", "wgrad_gateup", "router_bwd", "dW_r",
               "unpermute_bwd", "dx_router_term"]
EXPORTS = ["moe_create", "moe_destroy", "moe_workspace_bytes", "moe_workspace_find", "moe_status_string",
           "moe_poll_status", "moe_set_profiling", "moe_stage_times", "moe_forward", "moe_backward",
           "moe_e2e_device_bytes", "moe_step_host", "moe_router_wgrad_static", "moe_selftest_timeout",
           "moe_forward_inference", "moe_inference_workspace_bytes", "moe_backward_accumulate",
           "moe_lora_workspace_bytes", "moe_lora_forward", "moe_lora_backward",
           "moe_step_host_begin", "moe_step_host_end", "moe_kernel_launches", "moe_ctx_device",
           "moe_e2e_workspace_offset", "moe_ep_create", "moe_ep_send_workspace_bytes", "moe_ep_own_workspace_bytes",
           "moe_ep_workspace_find", "moe_ep_route", "moe_ep_plan", "moe_ep_dispatch", "moe_ep_expert_forward",
           "moe_ep_combine", "moe_ep_expert_backward", "moe_ep_expert_backward_accumulate", "moe_ep_router_backward",
           "moe_backward_accumulate_grouped", "moe_listwise_loss"]
EP_MAX_RANKS = 16  # MOE_EP_MAX_RANKS of include/moe.h
STATIC_MAX_DE = 262144  # MOE_STATIC_MAX_DE of include/moe.h


class MoEConfig(C.Structure):
    _fields_ = [("d", C.c_int32), ("E", C.c_int32), ("f", C.c_int32), ("top_k", C.c_int32), ("flags", C.c_int32)]


class MoEError(RuntimeError):
    pass


_lib = None


def load_library() -> C.CDLL:
    """Loads libmoe_b200.so built in-tree (python -m paper_2608_00916_b200.build).  Raises if absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise MoEError(f"{LIB_PATH} not found: build it with `python -m paper_2608_00916_b200.build`")
    lib = C.CDLL(LIB_PATH)
    vp, i64, sz = C.c_void_p, C.c_int64, C.c_size_t
    lib.moe_create.argtypes = [C.POINTER(MoEConfig), C.POINTER(vp)]
    lib.moe_create.restype = C.c_int
    lib.moe_destroy.argtypes = [vp]
    lib.moe_destroy.restype = None
    lib.moe_workspace_bytes.argtypes = [vp, i64]
    lib.moe_workspace_bytes.restype = sz
    lib.moe_workspace_find.argtypes = [vp, i64, C.c_char_p, C.POINTER(sz), C.POINTER(sz)]
    lib.moe_workspace_find.restype = C.c_int
    lib.moe_status_string.argtypes = [C.c_int]
    lib.moe_status_string.restype = C.c_char_p
    lib.moe_poll_status.argtypes = [vp, vp, vp]
    lib.moe_poll_status.restype = C.c_int
    lib.moe_set_profiling.argtypes = [vp, C.c_int]
    lib.moe_set_profiling.restype = C.c_int
    lib.moe_stage_times.argtypes = [vp, C.POINTER(C.c_float), C.POINTER(C.c_int32)]
    lib.moe_stage_times.restype = C.c_int
    lib.moe_forward.argtypes = [vp, i64] + [vp] * 14 + [vp, sz, vp]
    lib.moe_forward.restype = C.c_int
    lib.moe_forward_inference.argtypes = lib.moe_forward.argtypes
    lib.moe_forward_inference.restype = C.c_int
    lib.moe_inference_workspace_bytes.argtypes = [vp, i64]
    lib.moe_inference_workspace_bytes.restype = sz
    lib.moe_backward.argtypes = [vp, i64, vp, C.c_float] + [vp] * 11 + [vp, sz, vp]
    lib.moe_backward.restype = C.c_int
    lib.moe_backward_accumulate.argtypes = lib.moe_backward.argtypes
    lib.moe_backward_accumulate.restype = C.c_int
    lib.moe_backward_accumulate_grouped.argtypes = [vp, i64, vp, C.c_float] + [vp] * 11 + [C.c_int32, C.POINTER(vp), vp, sz, vp]
    lib.moe_backward_accumulate_grouped.restype = C.c_int
    lib.moe_step_host_begin.argtypes = [vp, C.c_int, i64, vp, vp, C.c_float, vp, vp, vp, vp, sz, vp]
    lib.moe_step_host_begin.restype = C.c_int
    lib.moe_step_host_end.argtypes = [vp, C.c_int]
    lib.moe_step_host_end.restype = C.c_int
    lib.moe_lora_workspace_bytes.argtypes = [vp, i64]
    lib.moe_lora_workspace_bytes.restype = sz
    lib.moe_lora_forward.argtypes = [vp, i64, C.c_int32, C.c_float] + [vp] * 16 + [vp, sz, vp]
    lib.moe_lora_forward.restype = C.c_int
    lib.moe_lora_backward.argtypes = [vp, i64, C.c_int32, C.c_float, vp, C.c_float] + [vp] * 17 + [vp, sz, vp]
    lib.moe_lora_backward.restype = C.c_int
    lib.moe_e2e_device_bytes.argtypes = [vp, i64]
    lib.moe_e2e_device_bytes.restype = sz
    lib.moe_e2e_workspace_offset.argtypes = [vp, i64]
    lib.moe_e2e_workspace_offset.restype = sz
    lib.moe_step_host.argtypes = [vp, i64, C.c_int] + [vp] * 6 + [C.c_float] + [vp] * 7 + [vp, sz, vp]
    lib.moe_step_host.restype = C.c_int
    lib.moe_kernel_launches.argtypes = []
    lib.moe_kernel_launches.restype = C.c_longlong
    lib.moe_ctx_device.argtypes = [vp]
    lib.moe_ctx_device.restype = C.c_int
    lib.moe_ep_create.argtypes = [C.POINTER(MoEConfig), C.c_int32, C.c_int32, i64, C.POINTER(vp)]
    lib.moe_ep_create.restype = C.c_int
    lib.moe_ep_send_workspace_bytes.argtypes = [vp, i64]
    lib.moe_ep_send_workspace_bytes.restype = sz
    lib.moe_ep_own_workspace_bytes.argtypes = [vp]
    lib.moe_ep_own_workspace_bytes.restype = sz
    lib.moe_ep_workspace_find.argtypes = [vp, i64, C.c_int, C.c_char_p, C.POINTER(sz), C.POINTER(sz)]
    lib.moe_ep_workspace_find.restype = C.c_int
    lib.moe_ep_route.argtypes = [vp, i64] + [vp] * 7 + [vp, sz, vp]
    lib.moe_ep_route.restype = C.c_int
    lib.moe_ep_plan.argtypes = [vp, i64, vp, vp, sz, vp, sz, vp]
    lib.moe_ep_plan.restype = C.c_int
    lib.moe_ep_dispatch.argtypes = [vp, i64, vp, C.c_int, C.POINTER(vp), vp, sz, vp]
    lib.moe_ep_dispatch.restype = C.c_int
    lib.moe_ep_expert_forward.argtypes = [vp, vp, vp, vp, vp, sz, vp]
    lib.moe_ep_expert_forward.restype = C.c_int
    lib.moe_ep_combine.argtypes = [vp, i64, C.POINTER(vp), vp, sz, vp, vp]
    lib.moe_ep_combine.restype = C.c_int
    lib.moe_ep_expert_backward.argtypes = [vp] + [vp] * 6 + [vp, sz, vp]
    lib.moe_ep_expert_backward.restype = C.c_int
    lib.moe_ep_expert_backward_accumulate.argtypes = [vp] + [vp] * 6 + [vp, sz, vp]
    lib.moe_ep_expert_backward_accumulate.restype = C.c_int
    lib.moe_ep_router_backward.argtypes = [vp, i64, C.c_float, vp, vp, C.POINTER(vp), vp, sz, vp, vp, vp, vp]
    lib.moe_ep_router_backward.restype = C.c_int
    lib.moe_listwise_loss.argtypes = [C.c_int32, i64, C.c_int32, vp, vp, C.c_float, C.c_float, vp, vp, vp]
    lib.moe_listwise_loss.restype = C.c_int
    lib.moe_selftest_timeout.argtypes = [vp, vp, vp]
    lib.moe_selftest_timeout.restype = C.c_int
    lib.moe_router_wgrad_static.argtypes = [i64, C.c_int32, C.c_int32, vp, vp, vp, vp]
    lib.moe_router_wgrad_static.restype = C.c_int
    _lib = lib
    return lib


def _check(lib, rc: int, what: str) -> None:
    if rc != 0:
        raise MoEError(f"{what}: {lib.moe_status_string(rc).decode()} ({rc})")


def kernel_launches() -> int:
    """Kernels the library has launched in this process so far."""
    return int(load_library().moe_kernel_launches())


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def listwise_loss(scores, teacher=None, s_temp: float = 1.0, t_temp: float = 1.0, want_grad: bool = True):
    """moe_listwise_loss on CUDA tensors: scores [n, G] fp32 (one row per query).  Without `teacher`: listwise
    cross-entropy with the positive at position 0; with teacher [n, G] fp32: temperature-scaled KL to the teacher's
    distribution.  Returns (loss [1] fp32, dloss/dscores [n, G] fp32 or None)."""
    import torch
    lib = load_library()
    assert scores.is_cuda and scores.dtype == torch.float32 and scores.dim() == 2 and scores.is_contiguous()
    n, G = scores.shape
    kind = 0
    if teacher is not None:
        assert teacher.is_cuda and teacher.dtype == torch.float32 and tuple(teacher.shape) == (n, G) and teacher.is_contiguous()
        kind = 1
    loss = torch.empty(1, dtype=torch.float32, device=scores.device)
    grad = torch.empty_like(scores) if want_grad else None
    _check(lib, lib.moe_listwise_loss(kind, n, G, _ptr(scores), _ptr(teacher), C.c_float(s_temp), C.c_float(t_temp),
                                      _ptr(loss), _ptr(grad), C.c_void_p(torch.cuda.current_stream().cuda_stream)),
           "moe_listwise_loss")
    return loss, grad


def router_wgrad_static(x, dl, dW_r=None):
    """dW_r = x^T dl through the entry point that allocates nothing inside the library (its scratch is a fixed
    array in the library image).  x: bf16 [T,d] CUDA tensor, dl: fp32 [T,E] CUDA tensor.  The output tensor is the
    caller's: pass dW_r (fp32 [d,E]) to reuse one, otherwise torch allocates it here, outside the library.
    Raises MoEError (unsupported) when d * E exceeds STATIC_MAX_DE."""
    import torch
    lib = load_library()
    T, d = x.shape
    E = dl.shape[1]
    assert x.dtype == torch.bfloat16 and dl.dtype == torch.float32 and x.is_contiguous() and dl.is_contiguous()
    assert dl.shape[0] == T
    if dW_r is None:
        dW_r = torch.empty(d, E, dtype=torch.float32, device=x.device)
    rc = lib.moe_router_wgrad_static(T, d, E, _ptr(x), _ptr(dl), _ptr(dW_r),
                                     C.c_void_p(torch.cuda.current_stream().cuda_stream))
    _check(lib, rc, "moe_router_wgrad_static")
    return dW_r


class MoELayer:
    """One MoE FFN layer shape (d, E, f, top_k) bound to the CUDA library.

    forward() / backward() take and return torch CUDA tensors (bf16 for activations and weights); the
    tensors are only carriers of device pointers."""

    def __init__(self, d: int, E: int, f: int, top_k: int, flags: int = 0):
        self.lib = load_library()
        self.d, self.E, self.f, self.k = d, E, f, top_k
        self.flags = flags
        cfg = MoEConfig(d, E, f, top_k, flags)
        h = C.c_void_p()
        _check(self.lib, self.lib.moe_create(C.byref(cfg), C.byref(h)), "moe_create")
        self.h = h
        self.ws = None
        self.T = None
        self._saved = None

    def __del__(self):
        try:
            if getattr(self, "h", None):
                self.lib.moe_destroy(self.h)
                self.h = None
        except Exception:
            pass

    # ---- workspace
    def workspace_bytes(self, T: int) -> int:
        return int(self.lib.moe_workspace_bytes(self.h, T))

    def inference_workspace_bytes(self, T: int) -> int:
        return int(self.lib.moe_inference_workspace_bytes(self.h, T))

    def find(self, T: int, name: str):
        off, n = C.c_size_t(), C.c_size_t()
        _check(self.lib, self.lib.moe_workspace_find(self.h, T, name.encode(), C.byref(off), C.byref(n)),
               f"moe_workspace_find({name})")
        return off.value, n.value

    def buffer(self, name: str, dtype):
        """View of an internal workspace buffer of the last forward call (for stage-by-stage tests)."""
        off, n = self.find(self.T, name)
        return self.ws[off:off + n].view(dtype)

    def _ensure_ws(self, T: int, inference: bool = False):
        import torch
        need = self.inference_workspace_bytes(T) if inference else self.workspace_bytes(T)
        if self.ws is None or self.ws.numel() < need:
            self.ws = torch.empty(max(need, 256), dtype=torch.uint8, device="cuda")
        self.T = T

    def _stream(self):
        import torch
        return C.c_void_p(torch.cuda.current_stream().cuda_stream)

    # ---- calls
    def forward(self, x, W_r, W_gate, W_up, W_down, b_r=None, logits_in=None, want_logits=False, want_perm=True,
                inference=False):
        """inference=True runs moe_forward_inference: no pre-activations are saved and backward() is not possible."""
        import torch
        T = x.shape[0]
        d, E, f, k = self.d, self.E, self.f, self.k
        assert x.dtype == torch.bfloat16 and tuple(x.shape) == (T, d) and x.is_contiguous()
        wr_dtype = torch.float32 if (self.flags & FLAG_ROUTER_FP32) else torch.bfloat16
        assert tuple(W_r.shape) == (d, E) and W_r.dtype == wr_dtype and W_r.is_contiguous()
        for w, shp in ((W_gate, (E, d, f)), (W_up, (E, d, f)), (W_down, (E, f, d))):
            assert tuple(w.shape) == shp and w.dtype == torch.bfloat16 and w.is_contiguous()
        self._ensure_ws(T, inference)
        dev = x.device
        out = {
            "y": torch.empty(T, d, dtype=torch.bfloat16, device=dev),
            "idx": torch.empty(T, k, dtype=torch.int32, device=dev),
            "gates": torch.empty(T, k, dtype=torch.float32, device=dev),
            "counts": torch.empty(E, dtype=torch.int32, device=dev),
            "perm": torch.empty(T * k, dtype=torch.int32, device=dev) if want_perm else None,
            "aux": torch.empty(1, dtype=torch.float32, device=dev),
            "logits": torch.empty(T, E, dtype=torch.float32, device=dev) if want_logits else None,
        }
        if b_r is not None:
            assert b_r.dtype == torch.float32 and b_r.numel() == E
        if logits_in is not None:
            assert logits_in.dtype == torch.float32 and tuple(logits_in.shape) == (T, E) and logits_in.is_contiguous()
        fn = self.lib.moe_forward_inference if inference else self.lib.moe_forward
        rc = fn(self.h, T, _ptr(x), _ptr(W_r), _ptr(b_r), _ptr(logits_in), _ptr(W_gate), _ptr(W_up), _ptr(W_down),
                _ptr(out["y"]), _ptr(out["idx"]), _ptr(out["gates"]), _ptr(out["counts"]), _ptr(out["perm"]),
                _ptr(out["aux"]), _ptr(out["logits"]), _ptr(self.ws), self.ws.numel(), self._stream())
        _check(self.lib, rc, "moe_forward")
        self._saved = None if inference else (x, W_r, W_gate, W_up, W_down)
        return out

    def backward(self, dy, d_aux: float, want_db: bool = False, grads=None):
        """Gradients for the last forward().  `grads` may carry preallocated output tensors."""
        import torch
        if self._saved is None:
            raise MoEError("backward() needs a preceding training forward()")
        x, W_r, W_gate, W_up, W_down = self._saved
        T = x.shape[0]
        d, E, f = self.d, self.E, self.f
        assert dy.dtype == torch.bfloat16 and tuple(dy.shape) == (T, d) and dy.is_contiguous()
        dev = x.device
        g = grads or {}

        def buf(name, shape, dtype):
            return g[name] if g.get(name) is not None else torch.empty(*shape, dtype=dtype, device=dev)

        out = {"dx": buf("dx", (T, d), torch.bfloat16), "dW_r": buf("dW_r", (d, E), torch.float32),
               "db_r": torch.empty(E, dtype=torch.float32, device=dev) if want_db else None,
               "dW_gate": buf("dW_gate", (E, d, f), torch.bfloat16), "dW_up": buf("dW_up", (E, d, f), torch.bfloat16),
               "dW_down": buf("dW_down", (E, f, d), torch.bfloat16)}
        rc = self.lib.moe_backward(self.h, T, _ptr(dy), C.c_float(d_aux), _ptr(x), _ptr(W_r), _ptr(W_gate), _ptr(W_up),
                                   _ptr(W_down), _ptr(out["dx"]), _ptr(out["dW_r"]), _ptr(out["db_r"]),
                                   _ptr(out["dW_gate"]), _ptr(out["dW_up"]), _ptr(out["dW_down"]), _ptr(self.ws),
                                   self.ws.numel(), self._stream())
        _check(self.lib, rc, "moe_backward")
        return out

    def backward_accumulate(self, dy, d_aux: float, acc, group_events=None):
        """Backward of the last forward() that adds the weight gradients into the fp32 tensors of `acc`
        (keys dW_r [d,E], dW_gate, dW_up [E,d,f], dW_down [E,f,d], optional db_r [E]); returns dx.
        group_events: 2 n torch.cuda.Event objects; the weight gradients then run in n ranges of experts and event g
        (n + g) is recorded when dW_down (dW_gate and dW_up) of range g is complete."""
        import torch
        if self._saved is None:
            raise MoEError("backward_accumulate() needs a preceding training forward()")
        x, W_r, W_gate, W_up, W_down = self._saved
        T = x.shape[0]
        for n, shp in (("dW_r", (self.d, self.E)), ("dW_gate", (self.E, self.d, self.f)), ("dW_up", (self.E, self.d, self.f)),
                       ("dW_down", (self.E, self.f, self.d))):
            assert acc[n].dtype == torch.float32 and tuple(acc[n].shape) == shp and acc[n].is_contiguous(), n
        dx = torch.empty(T, self.d, dtype=torch.bfloat16, device=x.device)
        if group_events is not None:
            n = len(group_events) // 2
            assert len(group_events) == 2 * n and n >= 1
            for ev in group_events:
                if ev.cuda_event == 0:  # torch creates the CUDA event lazily, at the first record
                    ev.record(torch.cuda.current_stream())
            evs = (C.c_void_p * (2 * n))(*[C.c_void_p(ev.cuda_event) for ev in group_events])
            rc = self.lib.moe_backward_accumulate_grouped(
                self.h, T, _ptr(dy), C.c_float(d_aux), _ptr(x), _ptr(W_r), _ptr(W_gate), _ptr(W_up), _ptr(W_down), _ptr(dx),
                _ptr(acc["dW_r"]), _ptr(acc.get("db_r")), _ptr(acc["dW_gate"]), _ptr(acc["dW_up"]), _ptr(acc["dW_down"]), n,
                evs, _ptr(self.ws), self.ws.numel(), self._stream())
            _check(self.lib, rc, "moe_backward_accumulate_grouped")
            return dx
        rc = self.lib.moe_backward_accumulate(self.h, T, _ptr(dy), C.c_float(d_aux), _ptr(x), _ptr(W_r), _ptr(W_gate),
                                              _ptr(W_up), _ptr(W_down), _ptr(dx), _ptr(acc["dW_r"]), _ptr(acc.get("db_r")),
                                              _ptr(acc["dW_gate"]), _ptr(acc["dW_up"]), _ptr(acc["dW_down"]),
                                              _ptr(self.ws), self.ws.numel(), self._stream())
        _check(self.lib, rc, "moe_backward_accumulate")
        return dx

    # ---- expert LoRA (frozen expert weights, rank-r adapters on fc1 and fc2)
    def lora_forward(self, x, W_r, W_gate, W_up, W_down, lora: dict, scale: float, b_r=None):
        """lora: dict of bf16 CUDA tensors A1 [E,d,r], B1_gate, B1_up [E,r,f], A2 [E,f,r], B2 [E,r,d]."""
        import torch
        T = x.shape[0]
        d, E, f, k = self.d, self.E, self.f, self.k
        r = lora["A1"].shape[2]
        for n, shp in (("A1", (E, d, r)), ("B1_gate", (E, r, f)), ("B1_up", (E, r, f)), ("A2", (E, f, r)), ("B2", (E, r, d))):
            assert tuple(lora[n].shape) == shp and lora[n].dtype == torch.bfloat16 and lora[n].is_contiguous(), n
        need = int(self.lib.moe_lora_workspace_bytes(self.h, T))
        if self.ws is None or self.ws.numel() < need:
            self.ws = torch.empty(max(need, 256), dtype=torch.uint8, device="cuda")
        self.T = T
        dev = x.device
        out = {"y": torch.empty(T, d, dtype=torch.bfloat16, device=dev),
               "idx": torch.empty(T, k, dtype=torch.int32, device=dev),
               "gates": torch.empty(T, k, dtype=torch.float32, device=dev),
               "counts": torch.empty(E, dtype=torch.int32, device=dev),
               "aux": torch.empty(1, dtype=torch.float32, device=dev)}
        rc = self.lib.moe_lora_forward(self.h, T, r, C.c_float(scale), _ptr(x), _ptr(W_r), _ptr(b_r), _ptr(W_gate),
                                       _ptr(W_up), _ptr(W_down), _ptr(lora["A1"]), _ptr(lora["B1_gate"]),
                                       _ptr(lora["B1_up"]), _ptr(lora["A2"]), _ptr(lora["B2"]), _ptr(out["y"]),
                                       _ptr(out["idx"]), _ptr(out["gates"]), _ptr(out["counts"]), _ptr(out["aux"]),
                                       _ptr(self.ws), self.ws.numel(), self._stream())
        _check(self.lib, rc, "moe_lora_forward")
        self._saved = None
        self._lora_saved = (x, W_r, W_gate, W_up, W_down, lora, scale)
        return out

    def lora_backward(self, dy, d_aux: float):
        import torch
        x, W_r, W_gate, W_up, W_down, lora, scale = self._lora_saved
        T = x.shape[0]
        r = lora["A1"].shape[2]
        dev = x.device
        out = {"dx": torch.empty(T, self.d, dtype=torch.bfloat16, device=dev),
               "dW_r": torch.empty(self.d, self.E, dtype=torch.float32, device=dev)}
        for n in ("A1", "B1_gate", "B1_up", "A2", "B2"):
            out["d" + n] = torch.empty_like(lora[n])
        rc = self.lib.moe_lora_backward(self.h, T, r, C.c_float(scale), _ptr(dy), C.c_float(d_aux), _ptr(x), _ptr(W_r),
                                        _ptr(W_gate), _ptr(W_up), _ptr(W_down), _ptr(lora["A1"]), _ptr(lora["B1_gate"]),
                                        _ptr(lora["B1_up"]), _ptr(lora["A2"]), _ptr(lora["B2"]), _ptr(out["dx"]),
                                        _ptr(out["dW_r"]), _ptr(out["dA1"]), _ptr(out["dB1_gate"]), _ptr(out["dB1_up"]),
                                        _ptr(out["dA2"]), _ptr(out["dB2"]), _ptr(self.ws), self.ws.numel(),
                                        self._stream())
        _check(self.lib, rc, "moe_lora_backward")
        return out

    def poll(self) -> None:
        """Synchronises and raises if a device-side bounded wait ran out."""
        _check(self.lib, self.lib.moe_poll_status(self.h, _ptr(self.ws), self._stream()), "device status")

    def step_host_begin(self, slot: int, T, dev_buf, host, d_aux: float):
        """Enqueues one pipelined host step for slot 0/1 (host: pinned x, dy in; y, aux, dx out); see step_host_end."""
        hp = lambda n: C.c_void_p(host[n].data_ptr())
        rc = self.lib.moe_step_host_begin(self.h, slot, T, hp("x"), hp("dy"), C.c_float(d_aux), hp("y"), hp("aux"),
                                          hp("dx"), _ptr(dev_buf), dev_buf.numel(), self._stream())
        _check(self.lib, rc, "moe_step_host_begin")

    def step_host_end(self, slot: int):
        _check(self.lib, self.lib.moe_step_host_end(self.h, slot), "moe_step_host_end")

    def selftest_timeout(self) -> None:
        """Launches the kernel whose bounded wait runs out (see moe_selftest_timeout); poll() then raises."""
        _check(self.lib, self.lib.moe_selftest_timeout(self.h, _ptr(self.ws), self._stream()), "moe_selftest_timeout")

    def set_profiling(self, on: bool) -> None:
        _check(self.lib, self.lib.moe_set_profiling(self.h, 1 if on else 0), "moe_set_profiling")

    def stage_times(self, acc=None):
        """Adds to `acc` the per-stage milliseconds summed over the forward+backward pairs recorded since the last
        call; returns (list of NUM_STAGES floats, number of pairs)."""
        arr = (C.c_float * NUM_STAGES)(*(acc or [0.0] * NUM_STAGES))
        n = C.c_int32(0)
        _check(self.lib, self.lib.moe_stage_times(self.h, arr, C.byref(n)), "moe_stage_times")
        return list(arr), n.value

    # ---- host-buffer step (end-to-end timing)
    def e2e_device_bytes(self, T: int) -> int:
        return int(self.lib.moe_e2e_device_bytes(self.h, T))

    def e2e_workspace_offset(self, T: int) -> int:
        return int(self.lib.moe_e2e_workspace_offset(self.h, T))

    def step_host(self, T, dev_buf, host, d_aux: float, copy_weights: bool):
        """host: dict of pinned CPU tensors x, W_r, W_gate, W_up, W_down, dy and outputs y, aux, dx, dW_r, dW_gate,
        dW_up, dW_down.  dev_buf: uint8 CUDA tensor of e2e_device_bytes(T)."""
        hp = lambda n: None if host.get(n) is None else C.c_void_p(host[n].data_ptr())
        rc = self.lib.moe_step_host(self.h, T, 1 if copy_weights else 0, hp("x"), hp("W_r"), hp("W_gate"), hp("W_up"),
                                    hp("W_down"), hp("dy"), C.c_float(d_aux), hp("y"), hp("aux"), hp("dx"), hp("dW_r"),
                                    hp("dW_gate"), hp("dW_up"), hp("dW_down"), _ptr(dev_buf), dev_buf.numel(),
                                    self._stream())
        _check(self.lib, rc, "moe_step_host")

"""ctypes binding of libmodse.so: the same calls as include/modse.h.

Argument marshalling only - every step of the layer runs in the library's CUDA
kernels.  PyTorch tensors are used as device buffers; their ``data_ptr()`` and
the current CUDA stream are handed to the C ABI.  There is no CPU fallback:
loading fails with an error if the shared library has not been built.
"""
from __future__ import annotations

import ctypes
import os

_PKG = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_PKG, "libmodse.so")

MODSE_OK = 0
MODSE_ERR_INVALID_ARG = 1
MODSE_ERR_UNSUPPORTED = 2
MODSE_ERR_WORKSPACE_TOO_SMALL = 3
MODSE_ERR_STATE = 4
MODSE_ERR_CUDA = 5
MODSE_ERR_DEVICE_TIMEOUT = 6
MODSE_ERR_DEVICE_BOUNDS = 7
MODSE_F32 = 0
MODSE_BF16 = 1
N_STAGES = 12
MODSE_FUSE_GATHER = 1
MODSE_FUSE_DG_ROWDOT = 2
MODSE_FUSE_SCATTER = 4
DEFAULT_TILE_PLAN = 0x3F3A         # every product on CTA pairs; fallback: products 1, 3, 4, 5 on one-CTA 256-row tiles
PAIR_SHIFT = 8                     # bit 8 + k of a plan: product k on 256-row tiles computed by a pair of CTAs


class ModseError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: status {status} ({status_string(status)})")


class _Weights(ctypes.Structure):
    _fields_ = [("w_router", ctypes.c_void_p), ("w_gate", ctypes.c_void_p), ("w_up", ctypes.c_void_p),
                ("w_down", ctypes.c_void_p)]


class _WGrads(ctypes.Structure):
    _fields_ = [("dw_router", ctypes.c_void_p), ("dw_gate", ctypes.c_void_p), ("dw_up", ctypes.c_void_p),
                ("dw_down", ctypes.c_void_p)]


_lib = None


def lib_path() -> str:
    return _LIB_PATH


def load():
    """Load libmodse.so (raises if it is missing: there is no other path)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise ImportError(f"{_LIB_PATH} not found: build it with `python -m paper_2409_12210_b200.build`")
    lib = ctypes.CDLL(_LIB_PATH)
    vp, ci, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
    ip = ctypes.POINTER(ctypes.c_int)
    lib.modse_create.restype = vp
    lib.modse_create.argtypes = [ci, ci, ip, ci]
    lib.modse_last_create_error.restype = ci
    lib.modse_destroy.restype = ci
    lib.modse_destroy.argtypes = [vp]
    lib.modse_check_pairs.restype = ci
    lib.modse_check_pairs.argtypes = [ip, ci, ip]
    lib.modse_status_string.restype = ctypes.c_char_p
    lib.modse_status_string.argtypes = [ci]
    lib.modse_workspace_bytes.restype = sz
    lib.modse_workspace_bytes.argtypes = [vp, ci, ci, ci]
    lib.modse_forward.restype = ci
    lib.modse_forward.argtypes = [vp, ci, ctypes.POINTER(_Weights), vp, ci, vp, vp, sz, ci, vp]
    lib.modse_backward.restype = ci
    lib.modse_backward.argtypes = [vp, ci, ctypes.POINTER(_Weights), vp, vp, ci, vp, ctypes.POINTER(_WGrads), vp, sz,
                                   vp]
    pp = ctypes.POINTER(ctypes.c_void_p)
    lib.modse_get_routing.restype = ci
    lib.modse_get_routing.argtypes = [vp, vp, ci, pp, pp, pp, pp, pp, pp, pp]
    lib.modse_get_gate_grads.restype = ci
    lib.modse_get_gate_grads.argtypes = [vp, vp, ci, pp, pp]
    lib.modse_check_device_status.restype = ci
    lib.modse_check_device_status.argtypes = [vp, vp, vp]
    lib.modse_last_launch_count.restype = ci
    lib.modse_last_launch_count.argtypes = [vp]
    lib.modse_route_static_scratch.restype = ci
    lib.modse_route_static_scratch.argtypes = [ci, ci, ci, ci, vp, vp, ci, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.modse_route_static_scratch_capacity.restype = sz
    lib.modse_route_static_scratch_status.restype = ci
    lib.modse_route_static_scratch_status.argtypes = [vp]
    lib.modse_aux_loss.restype = ci
    lib.modse_aux_loss.argtypes = [vp, vp, ci, ctypes.c_float, vp, vp, vp, vp]
    lib.modse_set_aux_loss.restype = ci
    lib.modse_set_aux_loss.argtypes = [vp, ctypes.c_float]
    lib.modse_set_noise_gate.restype = ci
    lib.modse_set_noise_gate.argtypes = [vp, vp, ctypes.c_float, ctypes.c_float]
    lib.modse_set_noise_grads.restype = ci
    lib.modse_set_noise_grads.argtypes = [vp, vp, vp]
    lib.modse_tune_forward.restype = ci
    lib.modse_tune_forward.argtypes = [vp, ci, ctypes.POINTER(_Weights), vp, ci, vp, vp, sz, ci, vp]
    lib.modse_get_tile_plan.restype = ci
    lib.modse_get_tile_plan.argtypes = [vp]
    lib.modse_set_tile_plan.restype = ci
    lib.modse_set_tile_plan.argtypes = [vp, ci]
    lib.modse_set_output_f32.restype = ci
    lib.modse_set_output_f32.argtypes = [vp, ci]
    lib.modse_stage_timing_begin.restype = ci
    lib.modse_stage_timing_begin.argtypes = [vp, ci]
    lib.modse_stage_timing_end.restype = ci
    lib.modse_stage_timing_end.argtypes = [vp, ctypes.POINTER(ctypes.c_float), ip]
    lib.modse_stage_name.restype = ctypes.c_char_p
    lib.modse_stage_name.argtypes = [ci]
    lib.modse_debug_set_default_tile_plan.restype = None
    lib.modse_debug_set_default_tile_plan.argtypes = [ci]
    lib.modse_debug_set_dynamic_tiles.restype = None
    lib.modse_debug_set_dynamic_tiles.argtypes = [ci]
    lib.modse_debug_set_epilogue_warps.restype = None
    lib.modse_debug_set_epilogue_warps.argtypes = [ci, ci, ci]
    lib.modse_debug_set_wait_limit_ms.restype = None
    lib.modse_debug_set_wait_limit_ms.argtypes = [ci]
    lib.modse_debug_skip_tile_loads.restype = None
    lib.modse_debug_skip_tile_loads.argtypes = [ci, ci]
    lib.modse_debug_workspace_offsets.restype = ci
    lib.modse_debug_workspace_offsets.argtypes = [vp, ci, ci, ci, ctypes.POINTER(sz), ctypes.POINTER(sz), ip]
    lib.modse_set_debug_checks.restype = ci
    lib.modse_set_debug_checks.argtypes = [vp, ci]
    lib.modse_set_fusion.restype = ci
    lib.modse_set_fusion.argtypes = [vp, ci]
    lib.modse_get_fusion.restype = ci
    lib.modse_get_fusion.argtypes = [vp]
    lib.modse_debug_use_fma_path.restype = None
    lib.modse_debug_use_fma_path.argtypes = [ci]
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load().modse_status_string(int(status)).decode()


def route_static_scratch(x, w_router, top_k: int):
    """Routing tables of a batch through modse_route_static_scratch: no workspace, the
    library's built-in scratch array is used.  Returns a dict of freshly created output
    tensors (the outputs are the caller's; only the scratch is the library's)."""
    import torch
    T, d = x.shape
    N = w_router.shape[0]
    dev = x.device
    out = {
        "topk_idx": torch.empty((T, top_k), dtype=torch.int32, device=dev),
        "topk_gate": torch.empty((T, top_k), dtype=torch.float32, device=dev),
        "counts": torch.empty(N, dtype=torch.int32, device=dev),
        "counts_slot": torch.empty((top_k, N), dtype=torch.int32, device=dev),
        "offsets": torch.empty(N + 1, dtype=torch.int32, device=dev),
        "row_of": torch.empty((T, top_k), dtype=torch.int32, device=dev),
        "token_of": torch.empty(T * top_k, dtype=torch.int32, device=dev),
    }
    st = load().modse_route_static_scratch(
        _dtype_code(x), d, N, top_k, x.data_ptr(), w_router.data_ptr(), T, out["topk_idx"].data_ptr(),
        out["topk_gate"].data_ptr(), out["counts"].data_ptr(), out["counts_slot"].data_ptr(),
        out["offsets"].data_ptr(), out["row_of"].data_ptr(), out["token_of"].data_ptr(),
        ctypes.c_void_p(torch.cuda.current_stream().cuda_stream))
    if st != MODSE_OK:
        raise ModseError(st, "modse_route_static_scratch")
    return out


def route_static_scratch_status() -> int:
    """Status word the last modse_route_static_scratch call on this device left (synchronises the stream)."""
    import torch
    return int(load().modse_route_static_scratch_status(ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)))


def stage_name(i: int) -> str:
    return load().modse_stage_name(int(i)).decode()


def debug_set_default_tile_plan(plan: int) -> None:
    load().modse_debug_set_default_tile_plan(int(plan))


def debug_set_dynamic_tiles(on: bool) -> None:
    load().modse_debug_set_dynamic_tiles(int(bool(on)))


def debug_set_epilogue_warps(mask_128: int = 0, mask_256: int = 5, mask_pair: int = 0) -> None:
    load().modse_debug_set_epilogue_warps(int(mask_128), int(mask_256), int(mask_pair))


def debug_set_wait_limit_ms(ms: int) -> None:
    load().modse_debug_set_wait_limit_ms(int(ms))


def debug_skip_tile_loads(product: int, tile: int) -> None:
    load().modse_debug_skip_tile_loads(int(product), int(tile))


def debug_use_fma_path(on: bool) -> None:
    load().modse_debug_use_fma_path(int(bool(on)))


def check_pairs(ffn_sizes):
    """(ok, pair_sum) for the adjacent-pair rule of Sec. 3.1, Eq. 5-6."""
    arr = (ctypes.c_int * len(ffn_sizes))(*ffn_sizes)
    out = ctypes.c_int(0)
    ok = load().modse_check_pairs(arr, len(ffn_sizes), ctypes.byref(out))
    return bool(ok), (out.value if ok else None)


def _dtype_code(t):
    import torch
    if t.dtype == torch.float32:
        return MODSE_F32
    if t.dtype == torch.bfloat16:
        return MODSE_BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


class ModseLayer:
    """Thin owner of a ``modse_layer_t``; methods mirror the C calls."""

    def __init__(self, d_model: int, ffn_sizes, top_k: int):
        lib = load()
        self.d_model, self.ffn_sizes, self.top_k = int(d_model), [int(h) for h in ffn_sizes], int(top_k)
        self.n_experts = len(self.ffn_sizes)
        arr = (ctypes.c_int * self.n_experts)(*self.ffn_sizes)
        self._h = lib.modse_create(self.d_model, self.n_experts, arr, self.top_k)
        if not self._h:
            raise ModseError(lib.modse_last_create_error(), "modse_create")

    def destroy(self):
        if getattr(self, "_h", None):
            load().modse_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    def workspace_bytes(self, dtype_code: int, n_tokens: int, save_for_backward: bool) -> int:
        return int(load().modse_workspace_bytes(self._h, dtype_code, n_tokens, int(save_for_backward)))

    def alloc_workspace(self, dtype, n_tokens: int, save_for_backward: bool, device="cuda"):
        import torch
        code = MODSE_F32 if dtype == torch.float32 else MODSE_BF16
        nbytes = self.workspace_bytes(code, n_tokens, save_for_backward)
        return torch.empty(max(nbytes, 256), dtype=torch.uint8, device=device)

    @staticmethod
    def _stream():
        import torch
        return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)

    def forward(self, w_router, w_gate, w_up, w_down, x, y, workspace, save_for_backward: bool):
        """Enqueue modse_forward on the current stream; tensors are device buffers
        laid out as include/modse.h states (w_down is [d, S])."""
        w = _Weights(w_router.data_ptr(), w_gate.data_ptr(), w_up.data_ptr(), w_down.data_ptr())
        st = load().modse_forward(self._h, _dtype_code(x), ctypes.byref(w), x.data_ptr(), x.shape[0], y.data_ptr(),
                                  workspace.data_ptr(), workspace.numel(), int(save_for_backward), self._stream())
        if st != MODSE_OK:
            raise ModseError(st, "modse_forward")

    def tune_forward(self, w_router, w_gate, w_up, w_down, x, y, workspace, save_for_backward: bool) -> int:
        """Time the kernel shapes of the forward products on this device (synchronises) and keep the fastest;
        returns the plan (see modse_get_tile_plan)."""
        w = _Weights(w_router.data_ptr(), w_gate.data_ptr(), w_up.data_ptr(), w_down.data_ptr())
        st = load().modse_tune_forward(self._h, _dtype_code(x), ctypes.byref(w), x.data_ptr(), x.shape[0],
                                       y.data_ptr(), workspace.data_ptr(), workspace.numel(),
                                       int(save_for_backward), self._stream())
        if st != MODSE_OK:
            raise ModseError(st, "modse_tune_forward")
        return self.tile_plan()

    def tile_plan(self) -> int:
        return int(load().modse_get_tile_plan(self._h))

    def set_tile_plan(self, plan: int) -> None:
        st = load().modse_set_tile_plan(self._h, int(plan))
        if st != MODSE_OK:
            raise ModseError(st, "modse_set_tile_plan")

    def backward(self, w_router, w_gate, w_up, w_down, x, dy, dx, dw_router, dw_gate, dw_up, dw_down, workspace):
        w = _Weights(w_router.data_ptr(), w_gate.data_ptr(), w_up.data_ptr(), w_down.data_ptr())
        g = _WGrads(dw_router.data_ptr(), dw_gate.data_ptr(), dw_up.data_ptr(), dw_down.data_ptr())
        st = load().modse_backward(self._h, _dtype_code(x), ctypes.byref(w), x.data_ptr(), dy.data_ptr(), x.shape[0],
                                   dx.data_ptr(), ctypes.byref(g), workspace.data_ptr(), workspace.numel(),
                                   self._stream())
        if st != MODSE_OK:
            raise ModseError(st, "modse_backward")

    @staticmethod
    def _view(ptr, workspace, count, dtype):
        off = ptr - workspace.data_ptr()
        return workspace[off:off + count * 4].view(dtype)

    def get_routing(self, workspace, n_tokens: int):
        """Views into the workspace: dict of topk_idx, topk_gate, counts, counts_slot,
        offsets, row_of, token_of (valid until the workspace is reused)."""
        import torch
        ptrs = [ctypes.c_void_p() for _ in range(7)]
        st = load().modse_get_routing(self._h, workspace.data_ptr(), n_tokens, *[ctypes.byref(p) for p in ptrs])
        if st != MODSE_OK:
            raise ModseError(st, "modse_get_routing")
        k, N, T = self.top_k, self.n_experts, n_tokens
        v = lambda i, n, dt: self._view(ptrs[i].value, workspace, n, dt)
        return {
            "topk_idx": v(0, T * k, torch.int32).view(T, k),
            "topk_gate": v(1, T * k, torch.float32).view(T, k),
            "counts": v(2, N, torch.int32),
            "counts_slot": v(3, k * N, torch.int32).view(k, N),
            "offsets": v(4, N + 1, torch.int32),
            "row_of": v(5, T * k, torch.int32).view(T, k),
            "token_of": v(6, T * k, torch.int32),
        }

    def get_gate_grads(self, workspace, n_tokens: int):
        import torch
        a, b = ctypes.c_void_p(), ctypes.c_void_p()
        st = load().modse_get_gate_grads(self._h, workspace.data_ptr(), n_tokens, ctypes.byref(a), ctypes.byref(b))
        if st != MODSE_OK:
            raise ModseError(st, "modse_get_gate_grads")
        T, k = n_tokens, self.top_k
        return (self._view(a.value, workspace, T * k, torch.float32).view(T, k),
                self._view(b.value, workspace, T * k, torch.float32).view(T, k))

    def check_device_status(self, workspace) -> int:
        return int(load().modse_check_device_status(self._h, workspace.data_ptr(), self._stream()))

    def set_debug_checks(self, on: bool) -> None:
        st = load().modse_set_debug_checks(self._h, int(bool(on)))
        if st != MODSE_OK:
            raise ModseError(st, "modse_set_debug_checks")

    def set_fusion(self, flags: int) -> None:
        st = load().modse_set_fusion(self._h, int(flags))
        if st != MODSE_OK:
            raise ModseError(st, "modse_set_fusion")

    def fusion(self) -> int:
        return int(load().modse_get_fusion(self._h))

    def debug_workspace_offsets(self, dtype_code: int, n_tokens: int, save_for_backward: bool):
        """(byte offset of prow_of, byte offset of the guard block behind topk_idx, padded rows)."""
        a, b, c = ctypes.c_size_t(0), ctypes.c_size_t(0), ctypes.c_int(0)
        st = load().modse_debug_workspace_offsets(self._h, dtype_code, n_tokens, int(save_for_backward),
                                                  ctypes.byref(a), ctypes.byref(b), ctypes.byref(c))
        if st != MODSE_OK:
            raise ModseError(st, "modse_debug_workspace_offsets")
        return int(a.value), int(b.value), int(c.value)

    def set_aux_loss(self, alpha: float) -> None:
        st = load().modse_set_aux_loss(self._h, float(alpha))
        if st != MODSE_OK:
            raise ModseError(st, "modse_set_aux_loss")

    def aux_loss(self, workspace, n_tokens: int, alpha: float):
        """(loss [1], f [N], P [N]) device tensors of the auxiliary load-balance loss (Eq. 7-10)."""
        import torch
        dev = workspace.device
        loss = torch.empty(1, dtype=torch.float32, device=dev)
        f = torch.empty(self.n_experts, dtype=torch.float32, device=dev)
        P = torch.empty(self.n_experts, dtype=torch.float32, device=dev)
        st = load().modse_aux_loss(self._h, workspace.data_ptr(), n_tokens, float(alpha), loss.data_ptr(),
                                   f.data_ptr(), P.data_ptr(), self._stream())
        if st != MODSE_OK:
            raise ModseError(st, "modse_aux_loss")
        return loss, f, P

    def set_noise_gate(self, w_noise, gamma: float = 0.0, eps: float = 0.0) -> None:
        """Second term of the router logits (Eq. 2): w_noise is a device tensor [N,d] in the layer's dtype
        that the caller keeps alive, or None to switch the term off."""
        self._w_noise = w_noise
        st = load().modse_set_noise_gate(self._h, w_noise.data_ptr() if w_noise is not None else None,
                                         float(gamma), float(eps))
        if st != MODSE_OK:
            raise ModseError(st, "modse_set_noise_gate")

    def set_noise_grads(self, dw_noise, dgamma) -> None:
        """Device tensors that backward fills: dw_noise [N,d] fp32, dgamma [1] fp32."""
        self._noise_grads = (dw_noise, dgamma)
        st = load().modse_set_noise_grads(self._h, dw_noise.data_ptr() if dw_noise is not None else None,
                                          dgamma.data_ptr() if dgamma is not None else None)
        if st != MODSE_OK:
            raise ModseError(st, "modse_set_noise_grads")

    def set_output_f32(self, on: bool) -> None:
        st = load().modse_set_output_f32(self._h, int(bool(on)))
        if st != MODSE_OK:
            raise ModseError(st, "modse_set_output_f32")

    def stage_timing_begin(self, max_calls: int) -> None:
        st = load().modse_stage_timing_begin(self._h, int(max_calls))
        if st != MODSE_OK:
            raise ModseError(st, "modse_stage_timing_begin")

    def stage_timing_end(self, max_calls: int):
        """[calls, N_STAGES] array of stage times in ms (-1: stage not run by that call)."""
        import numpy as np
        buf = (ctypes.c_float * (max_calls * N_STAGES))()
        n = ctypes.c_int(0)
        st = load().modse_stage_timing_end(self._h, buf, ctypes.byref(n))
        if st != MODSE_OK:
            raise ModseError(st, "modse_stage_timing_end")
        return np.ctypeslib.as_array(buf).reshape(max_calls, N_STAGES)[:n.value].copy()

    def last_launch_count(self) -> int:
        return int(load().modse_last_launch_count(self._h))


def pack_weights(inputs, device="cuda"):
    """Device tensors in the library's layouts from per-expert host arrays:
    w_router [N,d], w_gate/w_up [S,d], w_down [d,S] (experts side by side)."""
    import numpy as np
    import torch
    dt = torch.float32 if inputs.cfg.dtype == "f32" else torch.bfloat16
    to = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(device=device, dtype=dt)
    return (to(inputs.w_router), to(np.concatenate(inputs.w_gate, 0)), to(np.concatenate(inputs.w_up, 0)),
            to(np.concatenate(inputs.w_down, 1)))

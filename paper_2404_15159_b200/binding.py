"""ctypes binding of libmixlora.so: same names as include/mixlora.h, argument marshalling only.

PyTorch is used for device memory and streams.  There is no fallback of any kind: if the
library has not been built (`python -m paper_2404_15159_b200.build`) loading raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libmixlora.so")

MIXLORA_DTYPE_BF16 = 0
MIXLORA_DTYPE_FP32 = 1

STATUS_NAMES = {0: "MIXLORA_OK", 1: "MIXLORA_ERR_INVALID_ARG", 2: "MIXLORA_ERR_UNSUPPORTED",
                3: "MIXLORA_ERR_WORKSPACE", 4: "MIXLORA_ERR_CUDA", 5: "MIXLORA_ERR_DEVICE_TIMEOUT"}

EXPORTS = ("mixlora_limits", "mixlora_workspace_bytes", "mixlora_ffn_forward", "mixlora_aux_loss",
           "mixlora_ffn_backward", "mixlora_routing_view", "mixlora_device_status", "mixlora_gemm_bf16",
           "mixlora_status_string", "mixlora_stage_timing", "mixlora_stage_timing_read",
           "mixlora_dispatch_static", "mixlora_dispatch_static_max_tokens",
           "mixlora_multi_ffn_forward", "mixlora_multi_ffn_backward", "mixlora_layer_forward",
           "mixlora_layer_backward", "mixlora_lora_linear_workspace_bytes", "mixlora_lora_linear_forward",
           "mixlora_lora_linear_backward", "mixlora_lora_linear_status", "mixlora_ffn_backward_overlap",
           "mixlora_aux_stats", "mixlora_aux_loss_global", "mixlora_set_option", "mixlora_selftest_wait_timeout",
           "mixlora_dora_workspace_bytes", "mixlora_dora_ffn_forward", "mixlora_dora_ffn_backward")

MIXLORA_OPT_SERIAL = 0
MIXLORA_OPT_TC_SINGLE = 1


class mixlora_linear_shape_t(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("tokens", C.c_int32), ("d_in", C.c_int32), ("d_out", C.c_int32),
                ("rank", C.c_int32), ("lora_alpha", C.c_float), ("dtype", C.c_int32)]


class mixlora_shape_t(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("tokens", C.c_int32), ("d_model", C.c_int32), ("d_ff", C.c_int32),
                ("n_experts", C.c_int32), ("top_k", C.c_int32), ("rank", C.c_int32), ("lora_alpha", C.c_float),
                ("dtype", C.c_int32), ("renormalize", C.c_int32), ("aux_f_mode", C.c_int32)]


class mixlora_params_t(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("x", "w_gate", "w_up", "w_down", "w_router", "router_bias", "a_gate",
                                          "b_gate", "a_up", "b_up", "a_down", "b_down")]


class mixlora_grads_t(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("d_a_gate", "d_b_gate", "d_a_up", "d_b_up", "d_a_down", "d_b_down",
                                          "d_w_router", "d_router_bias", "d_x")] + [("accumulate", C.c_int32)]


class mixlora_dora_t(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("m_gate", "m_up", "m_down")]


class mixlora_dora_grads_t(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("d_m_gate", "d_m_up", "d_m_down")]


class mixlora_limits_t(C.Structure):
    _fields_ = [("max_experts", C.c_int32), ("max_top_k", C.c_int32), ("max_rank", C.c_int32)]


class MixLoraError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)} ({status_string(status)})")


def _load() -> C.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2404_15159_b200.build` "
                          "(there is no fallback path)")
    lib = C.CDLL(LIB_PATH)
    lib.mixlora_limits.argtypes = [C.POINTER(mixlora_limits_t)]
    lib.mixlora_limits.restype = None
    lib.mixlora_workspace_bytes.argtypes = [C.POINTER(mixlora_shape_t), C.c_int]
    lib.mixlora_workspace_bytes.restype = C.c_size_t
    lib.mixlora_ffn_forward.argtypes = [C.POINTER(mixlora_shape_t), C.POINTER(mixlora_params_t), C.c_void_p,
                                        C.c_void_p, C.c_size_t, C.c_void_p]
    lib.mixlora_ffn_forward.restype = C.c_int
    lib.mixlora_aux_loss.argtypes = [C.POINTER(mixlora_shape_t), C.c_void_p, C.c_float, C.c_void_p, C.c_void_p,
                                     C.c_void_p, C.c_void_p]
    lib.mixlora_aux_loss.restype = C.c_int
    lib.mixlora_ffn_backward.argtypes = [C.POINTER(mixlora_shape_t), C.POINTER(mixlora_params_t), C.c_void_p,
                                         C.c_float, C.c_void_p, C.c_size_t, C.POINTER(mixlora_grads_t), C.c_void_p]
    lib.mixlora_ffn_backward.restype = C.c_int
    lib.mixlora_routing_view.argtypes = [C.POINTER(mixlora_shape_t), C.c_void_p] + [C.POINTER(C.c_void_p)] * 6
    lib.mixlora_routing_view.restype = C.c_int
    lib.mixlora_device_status.argtypes = [C.c_void_p, C.POINTER(C.c_int32), C.c_void_p]
    lib.mixlora_device_status.restype = C.c_int
    lib.mixlora_gemm_bf16.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32,
                                      C.c_int32, C.c_void_p, C.c_void_p]
    lib.mixlora_gemm_bf16.restype = C.c_int
    lib.mixlora_stage_timing.argtypes = [C.c_int32]
    lib.mixlora_stage_timing.restype = C.c_int
    lib.mixlora_stage_timing_read.argtypes = [C.c_int32, C.POINTER(C.c_char_p), C.POINTER(C.c_float),
                                              C.POINTER(C.c_int64)]
    lib.mixlora_stage_timing_read.restype = C.c_int32
    lib.mixlora_dispatch_static.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p,
                                            C.c_void_p]
    lib.mixlora_dispatch_static.restype = C.c_int
    lib.mixlora_dispatch_static_max_tokens.argtypes = []
    lib.mixlora_dispatch_static_max_tokens.restype = C.c_int32
    lib.mixlora_multi_ffn_forward.argtypes = [C.c_int32, C.POINTER(mixlora_shape_t), C.POINTER(mixlora_params_t),
                                              C.POINTER(C.c_void_p), C.POINTER(C.c_void_p), C.POINTER(C.c_size_t),
                                              C.c_void_p]
    lib.mixlora_multi_ffn_forward.restype = C.c_int
    lib.mixlora_multi_ffn_backward.argtypes = [C.c_int32, C.POINTER(mixlora_shape_t), C.POINTER(mixlora_params_t),
                                               C.POINTER(C.c_void_p), C.POINTER(C.c_float), C.POINTER(C.c_void_p),
                                               C.POINTER(C.c_size_t), C.POINTER(mixlora_grads_t), C.c_void_p]
    lib.mixlora_multi_ffn_backward.restype = C.c_int
    lib.mixlora_layer_forward.argtypes = [C.POINTER(mixlora_shape_t), C.POINTER(mixlora_params_t), C.c_void_p, C.c_float,
                                          C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
    lib.mixlora_layer_forward.restype = C.c_int
    lib.mixlora_layer_backward.argtypes = [C.POINTER(mixlora_shape_t), C.POINTER(mixlora_params_t), C.c_void_p,
                                           C.c_float, C.c_void_p, C.c_void_p, C.c_void_p, C.c_float, C.c_void_p,
                                           C.c_size_t, C.POINTER(mixlora_grads_t), C.c_void_p]
    lib.mixlora_layer_backward.restype = C.c_int
    lib.mixlora_ffn_backward_overlap.argtypes = [C.POINTER(mixlora_shape_t), C.POINTER(mixlora_params_t), C.c_void_p,
                                                 C.c_float, C.c_void_p, C.c_size_t, C.POINTER(mixlora_grads_t),
                                                 C.c_void_p, C.c_void_p]
    lib.mixlora_ffn_backward_overlap.restype = C.c_int
    lib.mixlora_lora_linear_workspace_bytes.argtypes = [C.POINTER(mixlora_linear_shape_t)]
    lib.mixlora_lora_linear_workspace_bytes.restype = C.c_size_t
    lib.mixlora_lora_linear_forward.argtypes = [C.POINTER(mixlora_linear_shape_t)] + [C.c_void_p] * 6 + [C.c_size_t,
                                                                                                          C.c_void_p]
    lib.mixlora_lora_linear_forward.restype = C.c_int
    lib.mixlora_lora_linear_backward.argtypes = ([C.POINTER(mixlora_linear_shape_t)] + [C.c_void_p] * 6 +
                                                 [C.c_size_t, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p])
    lib.mixlora_lora_linear_backward.restype = C.c_int
    lib.mixlora_lora_linear_status.argtypes = [C.c_void_p, C.c_void_p]
    lib.mixlora_lora_linear_status.restype = C.c_int32
    lib.mixlora_aux_stats.argtypes = [C.POINTER(mixlora_shape_t), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    lib.mixlora_aux_stats.restype = C.c_int
    lib.mixlora_aux_loss_global.argtypes = [C.POINTER(mixlora_shape_t), C.c_void_p, C.c_float, C.c_void_p, C.c_void_p,
                                            C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    lib.mixlora_aux_loss_global.restype = C.c_int
    lib.mixlora_set_option.argtypes = [C.c_int32, C.c_int32]
    lib.mixlora_set_option.restype = C.c_int
    lib.mixlora_selftest_wait_timeout.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p]
    lib.mixlora_selftest_wait_timeout.restype = C.c_int
    lib.mixlora_dora_workspace_bytes.argtypes = [C.POINTER(mixlora_shape_t), C.c_int]
    lib.mixlora_dora_workspace_bytes.restype = C.c_size_t
    lib.mixlora_dora_ffn_forward.argtypes = [C.POINTER(mixlora_shape_t), C.POINTER(mixlora_params_t),
                                             C.POINTER(mixlora_dora_t), C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
    lib.mixlora_dora_ffn_forward.restype = C.c_int
    lib.mixlora_dora_ffn_backward.argtypes = [C.POINTER(mixlora_shape_t), C.POINTER(mixlora_params_t),
                                              C.POINTER(mixlora_dora_t), C.c_void_p, C.c_float, C.c_void_p, C.c_size_t,
                                              C.POINTER(mixlora_grads_t), C.POINTER(mixlora_dora_grads_t), C.c_void_p]
    lib.mixlora_dora_ffn_backward.restype = C.c_int
    lib.mixlora_status_string.argtypes = [C.c_int]
    lib.mixlora_status_string.restype = C.c_char_p
    return lib


lib = _load()


def status_string(status: int) -> str:
    return lib.mixlora_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != 0:
        raise MixLoraError(status, where)


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def make_shape(tokens, d_model, d_ff, n_experts, top_k, rank, lora_alpha, dtype=MIXLORA_DTYPE_BF16, renormalize=1,
               aux_f_mode=0) -> mixlora_shape_t:
    return mixlora_shape_t(C.sizeof(mixlora_shape_t), tokens, d_model, d_ff, n_experts, top_k, rank, float(lora_alpha),
                           dtype, renormalize, aux_f_mode)


def make_params(**tensors) -> mixlora_params_t:
    p = mixlora_params_t()
    for name, _ in mixlora_params_t._fields_:
        setattr(p, name, _ptr(tensors.get(name)))
    return p


def make_grads(accumulate=0, **tensors) -> mixlora_grads_t:
    g = mixlora_grads_t()
    for name, _ in mixlora_grads_t._fields_[:-1]:
        setattr(g, name, _ptr(tensors.get(name)))
    g.accumulate = int(accumulate)
    return g


def mixlora_limits() -> dict:
    out = mixlora_limits_t()
    lib.mixlora_limits(C.byref(out))
    return dict(max_experts=out.max_experts, max_top_k=out.max_top_k, max_rank=out.max_rank)


def mixlora_workspace_bytes(shape: mixlora_shape_t, for_backward: bool) -> int:
    return int(lib.mixlora_workspace_bytes(C.byref(shape), 1 if for_backward else 0))


def alloc_workspace(shape: mixlora_shape_t, for_backward: bool, device="cuda") -> torch.Tensor:
    n = mixlora_workspace_bytes(shape, for_backward)
    if n == 0:
        raise MixLoraError(1, "mixlora_workspace_bytes")
    return torch.empty(n, dtype=torch.uint8, device=device)


def mixlora_ffn_forward(shape, params, y, workspace, stream=None) -> None:
    _check(lib.mixlora_ffn_forward(C.byref(shape), C.byref(params), _ptr(y), _ptr(workspace),
                                   workspace.numel() if workspace is not None else 0, _stream(stream)),
           "mixlora_ffn_forward")


def mixlora_aux_loss(shape, workspace, coef, loss, F=None, P=None, stream=None) -> None:
    _check(lib.mixlora_aux_loss(C.byref(shape), _ptr(workspace), float(coef), _ptr(loss), _ptr(F), _ptr(P),
                                _stream(stream)), "mixlora_aux_loss")


def mixlora_aux_stats(shape, workspace, prob_sum, count, stream=None) -> None:
    """Un-normalised sums of Eq. 9 over this call's tokens (to be added over data-parallel shards)."""
    _check(lib.mixlora_aux_stats(C.byref(shape), _ptr(workspace), _ptr(prob_sum), _ptr(count), _stream(stream)),
           "mixlora_aux_stats")


def mixlora_aux_loss_global(shape, workspace, coef, prob_sum, count, total_tokens, loss, F=None, P=None,
                            stream=None) -> None:
    """Eq. 8-9 of the whole batch from the shards' added sums; the backward call that follows uses them too."""
    _check(lib.mixlora_aux_loss_global(C.byref(shape), _ptr(workspace), float(coef), _ptr(prob_sum), _ptr(count),
                                       int(total_tokens), _ptr(loss), _ptr(F), _ptr(P), _stream(stream)),
           "mixlora_aux_loss_global")


def mixlora_set_option(option: int, value: int) -> None:
    _check(lib.mixlora_set_option(int(option), int(value)), "mixlora_set_option")


def mixlora_selftest_wait_timeout(workspace, wait_rounds: int, stream=None) -> None:
    _check(lib.mixlora_selftest_wait_timeout(_ptr(workspace), int(wait_rounds), _stream(stream)),
           "mixlora_selftest_wait_timeout")


def mixlora_ffn_backward(shape, params, dy, aux_coef, workspace, grads, stream=None) -> None:
    _check(lib.mixlora_ffn_backward(C.byref(shape), C.byref(params), _ptr(dy), float(aux_coef), _ptr(workspace),
                                    workspace.numel() if workspace is not None else 0, C.byref(grads),
                                    _stream(stream)), "mixlora_ffn_backward")


def make_dora(m_gate, m_up, m_down) -> mixlora_dora_t:
    return mixlora_dora_t(_ptr(m_gate), _ptr(m_up), _ptr(m_down))


def make_dora_grads(d_m_gate=None, d_m_up=None, d_m_down=None) -> mixlora_dora_grads_t:
    return mixlora_dora_grads_t(_ptr(d_m_gate), _ptr(d_m_up), _ptr(d_m_down))


def alloc_dora_workspace(shape: mixlora_shape_t, for_backward: bool, device="cuda") -> torch.Tensor:
    n = int(lib.mixlora_dora_workspace_bytes(C.byref(shape), 1 if for_backward else 0))
    if n == 0:
        raise MixLoraError(1, "mixlora_dora_workspace_bytes")
    return torch.empty(n, dtype=torch.uint8, device=device)


def mixlora_dora_ffn_forward(shape, params, magnitudes, y, workspace, stream=None) -> None:
    _check(lib.mixlora_dora_ffn_forward(C.byref(shape), C.byref(params), C.byref(magnitudes), _ptr(y), _ptr(workspace),
                                        workspace.numel() if workspace is not None else 0, _stream(stream)),
           "mixlora_dora_ffn_forward")


def mixlora_dora_ffn_backward(shape, params, magnitudes, dy, aux_coef, workspace, grads, magnitude_grads,
                              stream=None) -> None:
    _check(lib.mixlora_dora_ffn_backward(C.byref(shape), C.byref(params), C.byref(magnitudes), _ptr(dy),
                                         float(aux_coef), _ptr(workspace),
                                         workspace.numel() if workspace is not None else 0, C.byref(grads),
                                         C.byref(magnitude_grads), _stream(stream)), "mixlora_dora_ffn_backward")


def mixlora_routing_view(shape, workspace) -> dict:
    """Zero-copy torch views of the routing that the last forward call left in `workspace`."""
    outs = [C.c_void_p() for _ in range(6)]
    _check(lib.mixlora_routing_view(C.byref(shape), _ptr(workspace), *[C.byref(o) for o in outs]),
           "mixlora_routing_view")
    base = workspace.data_ptr()
    T, k, N = shape.tokens, shape.top_k, shape.n_experts

    def view(ptr, nbytes, dtype, dims):
        off = ptr.value - base
        return workspace[off:off + nbytes].view(dtype).view(*dims)

    return dict(expert_idx=view(outs[0], T * k * 4, torch.int32, (T, k)),
                gates=view(outs[1], T * k * 4, torch.float32, (T, k)),
                perm=view(outs[2], T * k * 4, torch.int32, (T * k,)),
                seg_off=view(outs[3], (N + 1) * 4, torch.int32, (N + 1,)),
                low_margin=view(outs[4], T, torch.uint8, (T,)),
                probs=view(outs[5], T * N * 4, torch.float32, (T, N)))


def mixlora_device_status(workspace, stream=None) -> int:
    code = C.c_int32(0)
    _check(lib.mixlora_device_status(_ptr(workspace), C.byref(code), _stream(stream)), "mixlora_device_status")
    return int(code.value)


def mixlora_gemm_bf16(A, B, Cout, M, N, K, b_is_kn=False, status_word=None, stream=None) -> None:
    _check(lib.mixlora_gemm_bf16(_ptr(A), _ptr(B), _ptr(Cout), M, N, K, 1 if b_is_kn else 0, _ptr(status_word),
                                 _stream(stream)), "mixlora_gemm_bf16")


def mixlora_stage_timing(enable: bool) -> None:
    _check(lib.mixlora_stage_timing(1 if enable else 0), "mixlora_stage_timing")


def mixlora_stage_timing_read() -> dict:
    """{stage: (milliseconds, kernel launches)} accumulated since the last mixlora_stage_timing call."""
    n = 32
    names = (C.c_char_p * n)()
    ms = (C.c_float * n)()
    launches = (C.c_int64 * n)()
    cnt = lib.mixlora_stage_timing_read(n, names, ms, launches)
    return {names[i].decode(): (float(ms[i]), int(launches[i])) for i in range(min(cnt, n))}


def mixlora_dispatch_static(expert_idx, tokens, n_experts, top_k, perm, seg_off, stream=None) -> None:
    """Dispatch of slots to experts that needs no workspace: its scratch is a fixed array inside the
    library, so a caller that cannot allocate device memory can still use it (limits in mixlora.h)."""
    _check(lib.mixlora_dispatch_static(_ptr(expert_idx), tokens, n_experts, top_k, _ptr(perm), _ptr(seg_off),
                                       _stream(stream)), "mixlora_dispatch_static")


def mixlora_dispatch_static_max_tokens() -> int:
    return int(lib.mixlora_dispatch_static_max_tokens())


def _ptr_array(tensors):
    return (C.c_void_p * len(tensors))(*[_ptr(t) for t in tensors])


def mixlora_multi_ffn_forward(shapes, params, ys, workspaces, stream=None) -> None:
    """Forward of several adapters that share one frozen FFN (lists of equal length, one entry per adapter)."""
    n = len(shapes)
    _check(lib.mixlora_multi_ffn_forward(n, (mixlora_shape_t * n)(*shapes), (mixlora_params_t * n)(*params),
                                         _ptr_array(ys), _ptr_array(workspaces),
                                         (C.c_size_t * n)(*[w.numel() for w in workspaces]), _stream(stream)),
           "mixlora_multi_ffn_forward")


def mixlora_multi_ffn_backward(shapes, params, dys, aux_coefs, workspaces, grads, stream=None) -> None:
    n = len(shapes)
    _check(lib.mixlora_multi_ffn_backward(n, (mixlora_shape_t * n)(*shapes), (mixlora_params_t * n)(*params),
                                          _ptr_array(dys), (C.c_float * n)(*[float(a) for a in aux_coefs]),
                                          _ptr_array(workspaces), (C.c_size_t * n)(*[w.numel() for w in workspaces]),
                                          (mixlora_grads_t * n)(*grads), _stream(stream)),
           "mixlora_multi_ffn_backward")


def mixlora_layer_forward(shape, params, norm_weight, eps, xn, inv_rms, h, workspace, stream=None) -> None:
    """h = MixLoRA(RMSNorm(z)) + z with z = params.x; writes xn and inv_rms for the backward call."""
    _check(lib.mixlora_layer_forward(C.byref(shape), C.byref(params), _ptr(norm_weight), float(eps), _ptr(xn),
                                     _ptr(inv_rms), _ptr(h), _ptr(workspace),
                                     workspace.numel() if workspace is not None else 0, _stream(stream)),
           "mixlora_layer_forward")


def mixlora_layer_backward(shape, params, norm_weight, eps, xn, inv_rms, dh, aux_coef, workspace, grads,
                           stream=None) -> None:
    _check(lib.mixlora_layer_backward(C.byref(shape), C.byref(params), _ptr(norm_weight), float(eps), _ptr(xn),
                                      _ptr(inv_rms), _ptr(dh), float(aux_coef), _ptr(workspace),
                                      workspace.numel() if workspace is not None else 0, C.byref(grads),
                                      _stream(stream)), "mixlora_layer_backward")


def make_linear_shape(tokens, d_in, d_out, rank, lora_alpha, dtype=MIXLORA_DTYPE_BF16) -> mixlora_linear_shape_t:
    return mixlora_linear_shape_t(C.sizeof(mixlora_linear_shape_t), tokens, d_in, d_out, rank, float(lora_alpha), dtype)


def alloc_linear_workspace(shape) -> torch.Tensor:
    n = lib.mixlora_lora_linear_workspace_bytes(C.byref(shape))
    if n == 0:
        raise MixLoraError(1, "mixlora_lora_linear_workspace_bytes")
    return torch.empty(n, dtype=torch.uint8, device="cuda")


def mixlora_lora_linear_forward(shape, x, w, a, b, y, workspace, stream=None) -> None:
    """y = x W^T + s (x A^T) B^T (plain LoRA on a linear layer)."""
    _check(lib.mixlora_lora_linear_forward(C.byref(shape), _ptr(x), _ptr(w), _ptr(a), _ptr(b), _ptr(y), _ptr(workspace),
                                           workspace.numel() if workspace is not None else 0, _stream(stream)),
           "mixlora_lora_linear_forward")


def mixlora_lora_linear_backward(shape, x, w, a, b, dy, workspace, d_a=None, d_b=None, d_x=None, accumulate=0,
                                 stream=None) -> None:
    _check(lib.mixlora_lora_linear_backward(C.byref(shape), _ptr(x), _ptr(w), _ptr(a), _ptr(b), _ptr(dy),
                                            _ptr(workspace), workspace.numel() if workspace is not None else 0,
                                            _ptr(d_a), _ptr(d_b), _ptr(d_x), int(accumulate), _stream(stream)),
           "mixlora_lora_linear_backward")


def mixlora_lora_linear_status(workspace, stream=None) -> int:
    return int(lib.mixlora_lora_linear_status(_ptr(workspace), _stream(stream)))


def mixlora_ffn_backward_overlap(shape, params, dy, aux_coef, workspace, grads, ready_event, stream=None) -> None:
    """mixlora_ffn_backward that records `ready_event` (a torch.cuda.Event that has been recorded at least once, so
    that its handle exists) when the LoRA / router gradients are enqueued, before the input-gradient product."""
    handle = ready_event.cuda_event if ready_event is not None else None
    _check(lib.mixlora_ffn_backward_overlap(C.byref(shape), C.byref(params), _ptr(dy), float(aux_coef), _ptr(workspace),
                                            workspace.numel() if workspace is not None else 0, C.byref(grads),
                                            C.c_void_p(handle) if handle else None, _stream(stream)),
           "mixlora_ffn_backward_overlap")

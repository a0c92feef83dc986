"""ctypes binding of libtsp_mlp.so: same names as the C ABI, argument marshalling only.

Every step of the path runs inside the CUDA library.  If the library is missing the
functions raise; there is no fallback of any kind.  Tensors are torch CUDA tensors
(torch is used for device memory and streams only) or, for ``*_host`` calls, host
tensors / numpy arrays.
"""
from __future__ import annotations

import ctypes
import os

TSP_OK = 0
TSP_ERR_INVALID_ARG = -1
TSP_ERR_UNSUPPORTED_SHAPE = -2
TSP_ERR_UNSUPPORTED_DEVICE = -3
TSP_ERR_CUDA = -4
TSP_ERR_WORKSPACE = -5
TSP_ERR_DEVICE_TIMEOUT = -6
TSP_ERR_STATIC_LIMIT = -7
TSP_MLP_STATIC_SCRATCH_BYTES = 8 << 20
TSP_ACT_SILU = 0
TSP_ACT_GELU = 1
TSP_ACT_RELU = 2
TSP_WS_FORWARD = 0
TSP_WS_BACKWARD = 1

LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libtsp_mlp.so")

# name -> (restype, argtypes); mirrors include/tsp_mlp.h
_P = ctypes.c_void_p
SIGNATURES = {
    "tsp_mlp_plan": (ctypes.c_int, [ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.POINTER(_P)]),
    "tsp_mlp_options_default": (None, [_P]),
    "tsp_mlp_plan_ex": (ctypes.c_int, [ctypes.c_int, ctypes.c_int, ctypes.c_int, _P, ctypes.POINTER(_P)]),
    "tsp_mlp_plan_destroy": (ctypes.c_int, [_P]),
    "tsp_mlp_set_activation": (ctypes.c_int, [_P, ctypes.c_int]),
    "tsp_mlp_workspace_bytes": (ctypes.c_size_t, [_P, ctypes.c_int64, ctypes.c_int]),
    "tsp_mlp_workspace_bytes_host": (ctypes.c_size_t, [_P, ctypes.c_int64]),
    "tsp_mlp_set_workspace": (ctypes.c_int, [_P, _P, ctypes.c_size_t]),
    "tsp_mlp_forward": (ctypes.c_int, [_P, _P, _P, _P, _P, _P, ctypes.c_int64, ctypes.c_int, _P]),
    "tsp_mlp_saved_bytes": (ctypes.c_size_t, [_P, ctypes.c_int64]),
    "tsp_mlp_forward_save": (ctypes.c_int, [_P, _P, _P, _P, _P, _P, _P, ctypes.c_int64, ctypes.c_int, _P]),
    "tsp_mlp_backward_saved": (ctypes.c_int, [_P, _P, _P, _P, _P, _P, _P, _P, _P, _P, _P, ctypes.c_int64, ctypes.c_int, _P]),
    "tsp_mlp_forward_host": (ctypes.c_int, [_P, _P, _P, _P, _P, _P, ctypes.c_int64, ctypes.c_int, _P]),
    "tsp_mlp_backward": (ctypes.c_int, [_P, _P, _P, _P, _P, _P, _P, _P, _P, _P, ctypes.c_int64, ctypes.c_int, _P]),
    "tsp_mlp_workspace_bytes_staged": (ctypes.c_size_t, [_P, ctypes.c_int64]),
    "tsp_mlp_forward_staged": (ctypes.c_int, [_P, _P, _P, _P, _P, _P, ctypes.c_int64, ctypes.c_int, _P, _P]),
    "tsp_mlp_workspace_bytes_ring": (ctypes.c_size_t, [_P, ctypes.c_int64, ctypes.c_int]),
    "tsp_mlp_ring_step_backward_dx": (ctypes.c_int, [_P, _P, _P, _P, _P, _P, _P, ctypes.c_int64, ctypes.c_int, ctypes.c_int,
                                                     _P]),
    "tsp_mlp_ring_step_backward_dw": (ctypes.c_int, [_P, _P, _P, _P, _P, _P, ctypes.c_int64, ctypes.c_int, ctypes.c_int,
                                                     _P]),
    "tsp_mlp_ring_step_gate": (ctypes.c_int, [_P, _P, _P, _P, ctypes.c_int64, ctypes.c_int, ctypes.c_int, _P]),
    "tsp_mlp_ring_step_down": (ctypes.c_int, [_P, _P, _P, ctypes.c_int64, ctypes.c_int, ctypes.c_int, _P]),
    "tsp_mlp_workspace_bytes_ring_group": (ctypes.c_size_t, [_P, ctypes.c_int64, ctypes.c_int]),
    "tsp_mlp_ring_steps": (ctypes.c_int, [_P, _P, _P, _P, _P, ctypes.c_int64, ctypes.c_int, _P, ctypes.c_int64,
                                          ctypes.c_int, ctypes.c_int, _P]),
    "tsp_mlp_workspace_bytes_ring_group_backward": (ctypes.c_size_t, [_P, ctypes.c_int64, ctypes.c_int]),
    "tsp_mlp_ring_steps_backward_dx": (ctypes.c_int, [_P, _P, _P, _P, _P, ctypes.c_int64, ctypes.c_int, _P, _P,
                                                      ctypes.c_int64, ctypes.c_int, ctypes.c_int, _P]),
    "tsp_mlp_ring_steps_backward_dw": (ctypes.c_int, [_P, _P, _P, _P, _P, _P, ctypes.c_int64, ctypes.c_int, ctypes.c_int,
                                                      ctypes.c_int, ctypes.c_int, _P]),
    "tsp_mlp_ring_step": (ctypes.c_int, [_P, _P, _P, _P, _P, _P, ctypes.c_int64, ctypes.c_int, ctypes.c_int, _P]),
    "tsp_mlp_forward_static": (ctypes.c_int, [ctypes.c_int, ctypes.c_int, ctypes.c_int, _P, _P, _P, _P, _P,
                                              ctypes.c_int64, ctypes.POINTER(ctypes.c_int), _P]),
    "tsp_attn_plan": (ctypes.c_int, [ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.POINTER(_P)]),
    "tsp_attn_plan_destroy": (ctypes.c_int, [_P]),
    "tsp_attn_qkv_forward": (ctypes.c_int, [_P, _P, _P, _P, _P, _P, _P, _P, ctypes.c_int64, ctypes.c_int, _P]),
    "tsp_attn_out_forward": (ctypes.c_int, [_P, _P, _P, _P, ctypes.c_int64, ctypes.c_int, _P]),
    "tsp_attn_status": (ctypes.c_int, [_P]),
    "tsp_attn_profile_begin": (ctypes.c_int, [_P, ctypes.c_int]),
    "tsp_attn_profile_read": (ctypes.c_int, [_P, ctypes.c_int, ctypes.POINTER(ctypes.c_int),
                                             ctypes.POINTER(ctypes.c_float)]),
    "tsp_attn_qkv_backward": (ctypes.c_int, [_P] * 12 + [ctypes.c_int64, ctypes.c_int, _P]),
    "tsp_attn_out_backward": (ctypes.c_int, [_P] * 6 + [ctypes.c_int64, ctypes.c_int, _P]),
    "tsp_attn_profile_end": (ctypes.c_int, [_P]),
    "tsp_mlp_selftest_wait_expiry": (ctypes.c_int, [_P, ctypes.c_int, _P]),
    "tsp_mlp_status": (ctypes.c_int, [_P]),
    "tsp_mlp_error_string": (ctypes.c_char_p, [ctypes.c_int]),
    "tsp_mlp_last_cuda_error": (ctypes.c_int, [_P]),
    "tsp_mlp_ring_order": (ctypes.c_int, [_P, ctypes.POINTER(ctypes.c_int)]),
    "tsp_mlp_profile_begin": (ctypes.c_int, [_P, ctypes.c_int]),
    "tsp_mlp_profile_read": (ctypes.c_int, [_P, ctypes.c_int, ctypes.POINTER(ctypes.c_int), ctypes.POINTER(ctypes.c_float)]),
    "tsp_mlp_profile_end": (ctypes.c_int, [_P]),
    "tsp_mlp_kernels_per_call": (ctypes.c_int, [_P, ctypes.c_int]),
}

_lib = None


class TspError(RuntimeError):
    def __init__(self, code: int, where: str, detail: str = ""):
        self.code = code
        msg = f"{where}: {error_string(code)} ({code})"
        if detail:
            msg += f" [{detail}]"
        super().__init__(msg)


def load_library() -> ctypes.CDLL:
    """Load libtsp_mlp.so (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with __graft_entry__.build() "
                "(python -m paper_2604_26294_b200.build); there is no CPU fallback")
        lib = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype = res
            fn.argtypes = args
        _lib = lib
    return _lib


def tsp_mlp_error_string(code: int) -> str:
    return load_library().tsp_mlp_error_string(code).decode()


error_string = tsp_mlp_error_string


def _ptr(t) -> int:
    """Address of a torch tensor's / numpy array's first element; None -> 0."""
    if t is None:
        return 0
    if hasattr(t, "data_ptr"):
        return t.data_ptr()
    if hasattr(t, "ctypes"):
        return t.ctypes.data
    return int(t)


def _stream_handle(stream) -> int:
    if stream is None:
        import torch

        return torch.cuda.current_stream().cuda_stream
    if hasattr(stream, "cuda_stream"):
        return stream.cuda_stream
    return int(stream)


def _check(code: int, where: str, plan=None):
    if code != TSP_OK:
        detail = ""
        if plan is not None and code == TSP_ERR_CUDA:
            detail = f"cuda error {load_library().tsp_mlp_last_cuda_error(plan)}"
        raise TspError(code, where, detail)


# --------------------------------------------------------------------------- C ABI, same names
def tsp_mlp_plan(H: int, F: int, D: int):
    """Create a plan for hidden H, intermediate width F, D shards on the current device."""
    out = ctypes.c_void_p()
    _check(load_library().tsp_mlp_plan(H, F, D, ctypes.byref(out)), "tsp_mlp_plan")
    return out


class TspMlpOptions(ctypes.Structure):
    """Mirror of tsp_mlp_options_t (include/tsp_mlp.h); every field defaults to TSP_OPT_AUTO."""

    _fields_ = [("struct_bytes", ctypes.c_uint32)] + [(n, ctypes.c_int) for n in (
        "use_pairs", "gate_band", "gate_order", "down_group", "dx_group", "dw_group", "wide_mask", "pair_stages",
        "chunk_bands", "chunk_tiles", "dw_chunk_rounds", "phase_mask", "timeout_ms", "dynamic_tiles", "fuse_ring_steps", "tma_carry", "rank_pair_tiles", "overlap_launches")]


def tsp_mlp_options_default() -> TspMlpOptions:
    o = TspMlpOptions()
    load_library().tsp_mlp_options_default(ctypes.byref(o))
    return o


def tsp_mlp_plan_ex(H: int, F: int, D: int, options: TspMlpOptions | None = None, **fields):
    """tsp_mlp_plan with options: pass a TspMlpOptions, or the fields to change as keywords."""
    if options is None and fields:
        options = tsp_mlp_options_default()
    for k, v in fields.items():
        if k not in dict(TspMlpOptions._fields_):
            raise TypeError(f"tsp_mlp_options_t has no field {k!r}")
        setattr(options, k, v)
    out = ctypes.c_void_p()
    ref = ctypes.byref(options) if options is not None else None
    _check(load_library().tsp_mlp_plan_ex(H, F, D, ref, ctypes.byref(out)), "tsp_mlp_plan_ex")
    return out


def tsp_mlp_plan_destroy(plan) -> None:
    _check(load_library().tsp_mlp_plan_destroy(plan), "tsp_mlp_plan_destroy")


def tsp_mlp_set_activation(plan, activation: int) -> None:
    """Gate activation: TSP_ACT_SILU (default), TSP_ACT_GELU (erf form) or TSP_ACT_RELU."""
    _check(load_library().tsp_mlp_set_activation(plan, activation), "tsp_mlp_set_activation")


def tsp_mlp_workspace_bytes(plan, S: int, backward: int = TSP_WS_FORWARD) -> int:
    return int(load_library().tsp_mlp_workspace_bytes(plan, S, backward))


def tsp_mlp_workspace_bytes_host(plan, S: int) -> int:
    return int(load_library().tsp_mlp_workspace_bytes_host(plan, S))


def tsp_mlp_set_workspace(plan, buf, nbytes: int | None = None) -> None:
    if nbytes is None:
        nbytes = buf.numel() * buf.element_size()
    _check(load_library().tsp_mlp_set_workspace(plan, _ptr(buf), nbytes), "tsp_mlp_set_workspace")


def tsp_mlp_forward(plan, X, Wg, Wu, Wd, Y, S: int, D: int, stream=None) -> None:
    _check(load_library().tsp_mlp_forward(plan, _ptr(X), _ptr(Wg), _ptr(Wu), _ptr(Wd), _ptr(Y), S, D,
                                          _stream_handle(stream)), "tsp_mlp_forward", plan)


def tsp_mlp_forward_host(plan, X, Wg, Wu, Wd, Y, S: int, D: int, stream=None) -> None:
    _check(load_library().tsp_mlp_forward_host(plan, _ptr(X), _ptr(Wg), _ptr(Wu), _ptr(Wd), _ptr(Y), S, D,
                                               _stream_handle(stream)), "tsp_mlp_forward_host", plan)


def tsp_mlp_backward(plan, X, Wg, Wu, Wd, dY, dX, dWg, dWu, dWd, S: int, D: int, stream=None) -> None:
    _check(load_library().tsp_mlp_backward(plan, _ptr(X), _ptr(Wg), _ptr(Wu), _ptr(Wd), _ptr(dY), _ptr(dX),
                                           _ptr(dWg), _ptr(dWu), _ptr(dWd), S, D, _stream_handle(stream)),
           "tsp_mlp_backward", plan)


def tsp_mlp_workspace_bytes_staged(plan, S: int) -> int:
    return int(load_library().tsp_mlp_workspace_bytes_staged(plan, S))


def tsp_mlp_forward_staged(plan, X, Wg, Wu, Wd, Y, S: int, D: int, compute_stream=None, copy_stream=None) -> None:
    """Algorithm 2 step by step with the shard transfer emulated by copies on `copy_stream`."""
    _check(load_library().tsp_mlp_forward_staged(plan, _ptr(X), _ptr(Wg), _ptr(Wu), _ptr(Wd), _ptr(Y), S, D,
                                                 _stream_handle(compute_stream), _stream_handle(copy_stream)),
           "tsp_mlp_forward_staged", plan)


def tsp_mlp_workspace_bytes_ring(plan, S_loc: int, backward: int = TSP_WS_FORWARD) -> int:
    return int(load_library().tsp_mlp_workspace_bytes_ring(plan, S_loc, backward))


def tsp_mlp_ring_step(plan, X_p, Wg_k, Wu_k, Wd_k, Y_p, S_loc: int, t: int, D: int, stream=None) -> None:
    """One ring step of Algorithm 2 on one rank's tokens and the one shard it holds at step t."""
    _check(load_library().tsp_mlp_ring_step(plan, _ptr(X_p), _ptr(Wg_k), _ptr(Wu_k), _ptr(Wd_k), _ptr(Y_p), S_loc, t, D,
                                            _stream_handle(stream)), "tsp_mlp_ring_step", plan)


def tsp_mlp_ring_step_gate(plan, X_p, Wg_k, Wu_k, S_loc: int, t: int, D: int, stream=None) -> None:
    """First half of a ring step: the gate|up GEMM with the activation epilogue into the scratch buffer of step t."""
    _check(load_library().tsp_mlp_ring_step_gate(plan, _ptr(X_p), _ptr(Wg_k), _ptr(Wu_k), S_loc, t, D,
                                                 _stream_handle(stream)), "tsp_mlp_ring_step_gate", plan)


def tsp_mlp_ring_step_down(plan, Wd_k, Y_p, S_loc: int, t: int, D: int, stream=None) -> None:
    """Second half of a ring step: the shard's down projection added to the carried fp32 sum."""
    _check(load_library().tsp_mlp_ring_step_down(plan, _ptr(Wd_k), _ptr(Y_p), S_loc, t, D, _stream_handle(stream)),
           "tsp_mlp_ring_step_down", plan)


def tsp_mlp_workspace_bytes_ring_group(plan, S_loc: int, n_shards: int) -> int:
    return int(load_library().tsp_mlp_workspace_bytes_ring_group(plan, S_loc, n_shards))


def tsp_mlp_ring_steps(plan, X_p, Wg_first, Wu_first, Wd_first, shard_stride: int, n_shards: int, Y_p, S_loc: int,
                       t_first: int, D: int, stream=None) -> None:
    """n consecutive ring steps of one rank in one call; the n packed shards lie shard_stride elements apart."""
    _check(load_library().tsp_mlp_ring_steps(plan, _ptr(X_p), _ptr(Wg_first), _ptr(Wu_first), _ptr(Wd_first),
                                             shard_stride, n_shards, _ptr(Y_p), S_loc, t_first, D,
                                             _stream_handle(stream)), "tsp_mlp_ring_steps", plan)


def tsp_mlp_ring_step_backward_dx(plan, X_p, Wg_k, Wu_k, Wd_k, dY_p, dX_p, S_loc: int, t: int, D: int, stream=None) -> None:
    """Backward of one ring step, first part: A, dG, dU into the workspace and the carried dX sum."""
    _check(load_library().tsp_mlp_ring_step_backward_dx(plan, _ptr(X_p), _ptr(Wg_k), _ptr(Wu_k), _ptr(Wd_k), _ptr(dY_p),
                                                        _ptr(dX_p), S_loc, t, D, _stream_handle(stream)),
           "tsp_mlp_ring_step_backward_dx", plan)


def tsp_mlp_ring_step_backward_dw(plan, X_p, dY_p, dWg_k, dWu_k, dWd_k, S_loc: int, accumulate: int, D: int,
                                  stream=None) -> None:
    """Backward of one ring step, second part: this rank's contribution to the held shard's weight gradients."""
    _check(load_library().tsp_mlp_ring_step_backward_dw(plan, _ptr(X_p), _ptr(dY_p), _ptr(dWg_k), _ptr(dWu_k),
                                                        _ptr(dWd_k), S_loc, accumulate, D, _stream_handle(stream)),
           "tsp_mlp_ring_step_backward_dw", plan)


def tsp_mlp_workspace_bytes_ring_group_backward(plan, S_loc: int, n_shards: int) -> int:
    return int(load_library().tsp_mlp_workspace_bytes_ring_group_backward(plan, S_loc, n_shards))


def tsp_mlp_ring_steps_backward_dx(plan, X_p, Wg_first, Wu_first, Wd_first, shard_stride: int, n_shards: int, dY_p, dX_p,
                                   S_loc: int, t_first: int, D: int, stream=None) -> None:
    """Backward of n consecutive ring steps of one rank, all but the weight gradients (dA, A/dG/dU, carried dX sum)."""
    _check(load_library().tsp_mlp_ring_steps_backward_dx(plan, _ptr(X_p), _ptr(Wg_first), _ptr(Wu_first), _ptr(Wd_first),
                                                         shard_stride, n_shards, _ptr(dY_p), _ptr(dX_p), S_loc, t_first, D,
                                                         _stream_handle(stream)), "tsp_mlp_ring_steps_backward_dx", plan)


def tsp_mlp_ring_steps_backward_dw(plan, X_p, dY_p, dWg_k, dWu_k, dWd_k, S_loc: int, shard_in_group: int, n_shards: int,
                                   accumulate: int, D: int, stream=None) -> None:
    """Weight gradients of one shard of the group the preceding tsp_mlp_ring_steps_backward_dx call processed."""
    _check(load_library().tsp_mlp_ring_steps_backward_dw(plan, _ptr(X_p), _ptr(dY_p), _ptr(dWg_k), _ptr(dWu_k),
                                                         _ptr(dWd_k), S_loc, shard_in_group, n_shards, accumulate, D,
                                                         _stream_handle(stream)), "tsp_mlp_ring_steps_backward_dw", plan)


def tsp_mlp_forward_static(H: int, F: int, D: int, X, Wg, Wu, Wd, Y, S: int, timed_out=None, stream=None) -> None:
    """Forward pass that allocates nothing: for callers that cannot get device memory at call time.

    The intermediate lives in a fixed array inside the library (S*F*2 bytes <= TSP_MLP_STATIC_SCRATCH_BYTES).
    `timed_out`: optional ``ctypes.c_int`` filled (after a stream synchronize) with 0, or non-zero if a
    device-side wait expired.  Calls that overlap on the GPU race on the shared array.
    """
    ref = ctypes.byref(timed_out) if timed_out is not None else None
    _check(load_library().tsp_mlp_forward_static(H, F, D, _ptr(X), _ptr(Wg), _ptr(Wu), _ptr(Wd), _ptr(Y), S, ref,
                                                 _stream_handle(stream)), "tsp_mlp_forward_static")


def tsp_mlp_selftest_wait_expiry(plan, limit_ms: int = 20, stream=None) -> None:
    """Make one bounded device-side wait expire on purpose (sets the plan's status word; harmless)."""
    _check(load_library().tsp_mlp_selftest_wait_expiry(plan, limit_ms, _stream_handle(stream)),
           "tsp_mlp_selftest_wait_expiry", plan)


def tsp_mlp_saved_bytes(plan, S: int) -> int:
    return int(load_library().tsp_mlp_saved_bytes(plan, S))


def tsp_mlp_forward_save(plan, X, Wg, Wu, Wd, Y, saved, S: int, D: int, stream=None) -> None:
    """Forward that also keeps A, U*sigma'(G) and sigma(G) in `saved` for tsp_mlp_backward_saved."""
    _check(load_library().tsp_mlp_forward_save(plan, _ptr(X), _ptr(Wg), _ptr(Wu), _ptr(Wd), _ptr(Y), _ptr(saved), S, D,
                                               _stream_handle(stream)), "tsp_mlp_forward_save", plan)


def tsp_mlp_backward_saved(plan, X, Wg, Wu, Wd, dY, saved, dX, dWg, dWu, dWd, S: int, D: int, stream=None) -> None:
    """Backward from stored activations (no gate|up recomputation)."""
    _check(load_library().tsp_mlp_backward_saved(plan, _ptr(X), _ptr(Wg), _ptr(Wu), _ptr(Wd), _ptr(dY), _ptr(saved),
                                                 _ptr(dX), _ptr(dWg), _ptr(dWu), _ptr(dWd), S, D,
                                                 _stream_handle(stream)), "tsp_mlp_backward_saved", plan)


def tsp_mlp_status(plan) -> int:
    """Device status word as a status code (TSP_OK or TSP_ERR_DEVICE_TIMEOUT); does not raise."""
    return int(load_library().tsp_mlp_status(plan))


def tsp_mlp_last_cuda_error(plan) -> int:
    return int(load_library().tsp_mlp_last_cuda_error(plan))


def tsp_mlp_ring_order(plan, D: int):
    table = (ctypes.c_int * (D * D))()
    _check(load_library().tsp_mlp_ring_order(plan, table), "tsp_mlp_ring_order")
    return [[table[r * D + t] for t in range(D)] for r in range(D)]


def tsp_mlp_profile_begin(plan, max_calls: int) -> None:
    _check(load_library().tsp_mlp_profile_begin(plan, max_calls), "tsp_mlp_profile_begin", plan)


def tsp_mlp_profile_read(plan, call_index: int):
    n = ctypes.c_int()
    ms = (ctypes.c_float * 8)()
    _check(load_library().tsp_mlp_profile_read(plan, call_index, ctypes.byref(n), ms), "tsp_mlp_profile_read", plan)
    return [float(ms[i]) for i in range(n.value)]


def tsp_mlp_profile_end(plan) -> None:
    _check(load_library().tsp_mlp_profile_end(plan), "tsp_mlp_profile_end")


def tsp_mlp_kernels_per_call(plan, backward: int = TSP_WS_FORWARD) -> int:
    return int(load_library().tsp_mlp_kernels_per_call(plan, backward))


# --------------------------------------------------------------------------- include/tsp_attn.h, same names
def tsp_attn_plan(H: int, Hq: int, Hkv: int, D: int):
    """Plan for the projection GEMMs of TSP attention: hidden H, query width Hq, key/value width Hkv, D shards."""
    out = ctypes.c_void_p()
    _check(load_library().tsp_attn_plan(H, Hq, Hkv, D, ctypes.byref(out)), "tsp_attn_plan")
    return out


def tsp_attn_plan_destroy(plan) -> None:
    _check(load_library().tsp_attn_plan_destroy(plan), "tsp_attn_plan_destroy")


def tsp_attn_qkv_forward(plan, X, Wq, Wk, Wv, Q, K, V, S: int, D: int, stream=None) -> None:
    _check(load_library().tsp_attn_qkv_forward(plan, _ptr(X), _ptr(Wq), _ptr(Wk), _ptr(Wv), _ptr(Q), _ptr(K), _ptr(V),
                                               S, D, _stream_handle(stream)), "tsp_attn_qkv_forward")


def tsp_attn_out_forward(plan, A, Wo, Y, S: int, D: int, stream=None) -> None:
    _check(load_library().tsp_attn_out_forward(plan, _ptr(A), _ptr(Wo), _ptr(Y), S, D, _stream_handle(stream)),
           "tsp_attn_out_forward")


def tsp_attn_status(plan) -> int:
    return int(load_library().tsp_attn_status(plan))


def tsp_attn_profile_begin(plan, max_calls: int) -> None:
    _check(load_library().tsp_attn_profile_begin(plan, max_calls), "tsp_attn_profile_begin")


def tsp_attn_profile_read(plan, call_index: int) -> list[float]:
    """Kernel durations (ms) of one recorded call: one value for a forward call, two for a backward call."""
    n = ctypes.c_int()
    ms = (ctypes.c_float * 8)()
    _check(load_library().tsp_attn_profile_read(plan, call_index, ctypes.byref(n), ms), "tsp_attn_profile_read")
    return [float(ms[i]) for i in range(n.value)]


def tsp_attn_qkv_backward(plan, X, Wq, Wk, Wv, dQ, dK, dV, dX, dWq, dWk, dWv, S: int, D: int, stream=None) -> None:
    _check(load_library().tsp_attn_qkv_backward(plan, _ptr(X), _ptr(Wq), _ptr(Wk), _ptr(Wv), _ptr(dQ), _ptr(dK),
                                                _ptr(dV), _ptr(dX), _ptr(dWq), _ptr(dWk), _ptr(dWv), S, D,
                                                _stream_handle(stream)), "tsp_attn_qkv_backward")


def tsp_attn_out_backward(plan, A, Wo, dY, dA, dWo, S: int, D: int, stream=None) -> None:
    _check(load_library().tsp_attn_out_backward(plan, _ptr(A), _ptr(Wo), _ptr(dY), _ptr(dA), _ptr(dWo), S, D,
                                                _stream_handle(stream)), "tsp_attn_out_backward")


def tsp_attn_profile_end(plan) -> None:
    _check(load_library().tsp_attn_profile_end(plan), "tsp_attn_profile_end")

"""ctypes binding of libimpact.so: the same calls as include/impact.h, by the same names.

Argument marshalling only -- every step of the path runs in the CUDA library.  torch is
used for device memory and streams.  There is no fallback: a missing library, a missing
GPU or a non-zero status raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libimpact.so")

OK = 0
ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE_TOO_SMALL, ERR_EMPTY, ERR_FULL, ERR_CUDA = -1, -2, -3, -4, -5, -6
DTYPE_F32, DTYPE_BF16 = 0, 1
IS_TARGET_OVER_WORKER, IS_LEARNER_OVER_WORKER, IS_NONE = 0, 1, 2
OBJECTIVE_CLIPPED_SURROGATE, OBJECTIVE_VTRACE_PG = 0, 1
RATIO_R3, RATIO_R1, RATIO_R2 = 0, 1, 2
SAMPLE_UNIFORM, SAMPLE_ROUND_ROBIN = 0, 1
SRC_DEVICE, SRC_HOST = 0, 1
NUM_TERMS = 8
TERM_NAMES = ("total", "policy", "value", "entropy", "kl", "clip_frac", "rho_trunc_frac", "mean_ratio")

EXPORTS = (
    "impact_version", "impact_status_string", "impact_last_cuda_error",
    "impact_loss_workspace_bytes", "impact_loss_workspace_init", "impact_loss_fwd_bwd",
    "impact_loss_fwd_bwd_gaussian", "impact_buffer_storage_bytes", "impact_buffer_create",
    "impact_buffer_destroy", "impact_buffer_push", "impact_buffer_sample", "impact_buffer_append",
    "impact_buffer_slot_ptr", "impact_buffer_live", "impact_buffer_state_bytes",
    "impact_buffer_export_state", "impact_buffer_import_state", "impact_gather_rows",
    "impact_loss_fwd_bwd_static_scratch", "impact_loss_fwd_bwd_call", "impact_loss_workspace_status",
    "impact_set_option", "impact_get_option", "impact_loss_static_scratch_status", "impact_stream_copy",
    "impact_buffer_device_begin", "impact_buffer_device_end", "impact_buffer_device_step",
    "impact_buffer_device_events",
)
OPT_EARLY_PREFETCH, OPT_PREFETCH_BYTES, OPT_WINDOW_BYTES = 0, 1, 2


class ImpactError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(what)


class impact_coefficients(ctypes.Structure):
    _fields_ = [("vf_coef", ctypes.c_float), ("ent_coef", ctypes.c_float), ("kl_coef", ctypes.c_float),
                ("lambda_", ctypes.c_float), ("rho_tw", ctypes.c_float), ("is_source", ctypes.c_int32),
                ("ratio_mode", ctypes.c_int32), ("dlogits_dtype", ctypes.c_int32),
                ("objective", ctypes.c_int32), ("global_steps", ctypes.c_int64)]


class impact_loss_call(ctypes.Structure):
    _fields_ = [("learner_logits", ctypes.c_void_p), ("target_logits", ctypes.c_void_p),
                ("worker_logp", ctypes.c_void_p), ("actions", ctypes.c_void_p), ("rewards", ctypes.c_void_p),
                ("discounts", ctypes.c_void_p), ("values", ctypes.c_void_p), ("bootstrap_values", ctypes.c_void_p),
                ("rho_bar", ctypes.c_float), ("c_bar", ctypes.c_float), ("clip_eps", ctypes.c_float),
                ("logits_dtype", ctypes.c_int32), ("coef", impact_coefficients), ("A", ctypes.c_int32),
                ("B", ctypes.c_int64), ("T", ctypes.c_int64), ("loss_terms", ctypes.c_void_p),
                ("dlogits", ctypes.c_void_p), ("dvalues", ctypes.c_void_p), ("vtarget", ctypes.c_void_p),
                ("advantage", ctypes.c_void_p), ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t),
                ("target_logits_copy", ctypes.c_void_p), ("inputs_on_device", ctypes.c_void_p)]


class impact_ring_field_map(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("actions", "rewards", "discounts", "worker_logp", "target_logits")]


class impact_loss_inputs(ctypes.Structure):
    """Layout of the record impact_buffer_device_step writes (device memory; here only for its size and for
    reading one back in tests)."""
    _fields_ = [(n, ctypes.c_void_p) for n in ("learner_logits", "target_logits", "worker_logp", "actions", "rewards",
                                               "discounts", "values", "bootstrap_values", "target_logits_copy")] + \
               [(n, ctypes.c_int32) for n in ("status", "slot", "k_before", "pad")]


_lib = None
_vp, _i32, _i64, _f32, _sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_float, ctypes.c_size_t


def load_library() -> ctypes.CDLL:
    """Loads libimpact.so; raises if it has not been built (there is no other code path)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_1912_00167_b200.build`")
    lib = ctypes.CDLL(LIB_PATH)
    lib.impact_version.restype = _i32
    lib.impact_status_string.restype = ctypes.c_char_p
    lib.impact_status_string.argtypes = [_i32]
    lib.impact_last_cuda_error.restype = _i32
    lib.impact_loss_workspace_bytes.restype = _sz
    lib.impact_loss_workspace_bytes.argtypes = [_i64, _i64]
    lib.impact_loss_workspace_init.restype = _i32
    lib.impact_loss_workspace_init.argtypes = [_vp, _sz, _vp]
    lib.impact_loss_fwd_bwd.restype = _i32
    lib.impact_loss_fwd_bwd.argtypes = [_vp] * 8 + [_f32] * 3 + [ctypes.POINTER(impact_coefficients), _i64, _i64,
                                                               _i32, _i32] + [_vp] * 6 + [_sz, _vp]
    lib.impact_loss_workspace_status.restype = _i32
    lib.impact_loss_workspace_status.argtypes = [_vp, _sz, ctypes.POINTER(_i32), _vp]
    lib.impact_loss_fwd_bwd_call.restype = _i32
    lib.impact_loss_fwd_bwd_call.argtypes = [ctypes.POINTER(impact_loss_call), _vp]
    lib.impact_loss_fwd_bwd_static_scratch.restype = _i32
    lib.impact_loss_fwd_bwd_static_scratch.argtypes = [_vp] * 8 + [_f32] * 3 + [
        ctypes.POINTER(impact_coefficients), _i64, _i64, _i32, _i32] + [_vp] * 5 + [_vp]
    lib.impact_loss_fwd_bwd_gaussian.restype = _i32
    lib.impact_loss_fwd_bwd_gaussian.argtypes = [_vp] * 10 + [_f32] * 3 + [ctypes.POINTER(impact_coefficients),
                                                                         _i64, _i64, _i32] + [_vp] * 7 + [_sz, _vp]
    lib.impact_buffer_storage_bytes.restype = _sz
    lib.impact_buffer_storage_bytes.argtypes = [_i32, _i32, ctypes.POINTER(_sz)]
    lib.impact_buffer_create.restype = _i32
    lib.impact_buffer_create.argtypes = [_i32, _i32, _i32, ctypes.POINTER(_sz), ctypes.c_uint64, _i32, _vp,
                                         ctypes.POINTER(_vp)]
    lib.impact_buffer_destroy.restype = _i32
    lib.impact_buffer_destroy.argtypes = [_vp]
    lib.impact_buffer_push.restype = _i32
    lib.impact_buffer_push.argtypes = [_vp, ctypes.POINTER(_vp), _i32, ctypes.POINTER(_i32), _vp]
    lib.impact_buffer_sample.restype = _i32
    lib.impact_buffer_sample.argtypes = [_vp, ctypes.POINTER(_i32), ctypes.POINTER(_i32), ctypes.POINTER(_vp), _vp]
    lib.impact_buffer_append.restype = _i32
    lib.impact_buffer_append.argtypes = [_vp, _i32, _i32, _vp, _vp]
    lib.impact_buffer_slot_ptr.restype = _vp
    lib.impact_buffer_slot_ptr.argtypes = [_vp, _i32, _i32]
    lib.impact_buffer_live.restype = _i32
    lib.impact_buffer_live.argtypes = [_vp]
    lib.impact_buffer_state_bytes.restype = _sz
    lib.impact_buffer_state_bytes.argtypes = [_vp]
    lib.impact_buffer_export_state.restype = _i32
    lib.impact_buffer_export_state.argtypes = [_vp, _vp, _sz]
    lib.impact_buffer_import_state.restype = _i32
    lib.impact_buffer_import_state.argtypes = [_vp, _vp, _sz]
    lib.impact_gather_rows.restype = _i32
    lib.impact_gather_rows.argtypes = [_vp, _vp, _i64, _i64, _sz, _vp, _vp]
    lib.impact_loss_static_scratch_status.restype = _i32
    lib.impact_loss_static_scratch_status.argtypes = [ctypes.POINTER(_i32), _i32, _vp]
    lib.impact_buffer_device_begin.restype = _i32
    lib.impact_buffer_device_begin.argtypes = [_vp, _vp]
    lib.impact_buffer_device_end.restype = _i32
    lib.impact_buffer_device_end.argtypes = [_vp, _vp]
    lib.impact_buffer_device_step.restype = _i32
    lib.impact_buffer_device_step.argtypes = [_vp, ctypes.POINTER(impact_ring_field_map), _vp, _vp, _vp, _vp, _i32, _vp, _vp]
    lib.impact_buffer_device_events.restype = _i32
    lib.impact_buffer_device_events.argtypes = [_vp, ctypes.POINTER(_i32), _i32, ctypes.POINTER(_i32), _vp]
    lib.impact_stream_copy.restype = _i32
    lib.impact_stream_copy.argtypes = [_vp, _sz, _vp, _sz, _vp]
    lib.impact_set_option.restype = _i32
    lib.impact_set_option.argtypes = [_i32, _i64]
    lib.impact_get_option.restype = _i64
    lib.impact_get_option.argtypes = [_i32]
    _lib = lib
    return lib


def _check(status: int, what: str, allow=()) -> int:
    if status == OK or status in allow:
        return status
    lib = load_library()
    msg = lib.impact_status_string(status).decode()
    if status == ERR_CUDA:
        msg += f" (cudaError {lib.impact_last_cuda_error()})"
    raise ImpactError(status, f"{what}: {msg}")


def impact_version() -> int:
    return load_library().impact_version()


def impact_status_string(status: int) -> str:
    return load_library().impact_status_string(status).decode()


def impact_set_option(option: int, value: int) -> None:
    _check(load_library().impact_set_option(option, value), "impact_set_option")


def impact_get_option(option: int) -> int:
    return load_library().impact_get_option(option)


def _dev(t: torch.Tensor | None, dtype, shape, name: str, optional: bool = False) -> int | None:
    """Device pointer of a dense CUDA tensor after checking dtype and shape."""
    if t is None:
        if optional:
            return None
        raise ValueError(f"{name} is required")
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor (there is no CPU path)")
    if t.dtype != dtype or tuple(t.shape) != tuple(shape) or not t.is_contiguous():
        raise ValueError(f"{name}: expected contiguous {dtype} {tuple(shape)}, got {t.dtype} {tuple(t.shape)}")
    return t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


@dataclass
class Coefficients:
    """Host-side mirror of `impact_coefficients` plus the three scalars of the call."""

    rho_bar: float = 1.0
    c_bar: float = 1.0
    clip_eps: float = 0.2
    vf_coef: float = 0.5
    ent_coef: float = 0.01
    kl_coef: float = 0.0
    lam: float = 1.0
    rho_tw: float = 1.0
    is_source: int = IS_TARGET_OVER_WORKER
    ratio_mode: int = RATIO_R3
    objective: int = OBJECTIVE_CLIPPED_SURROGATE
    global_steps: int = 0  # steps of the whole train batch when it is split over several calls; 0 = this call's B*T

    def c_struct(self, dlogits_dtype: int) -> impact_coefficients:
        return impact_coefficients(self.vf_coef, self.ent_coef, self.kl_coef, self.lam, self.rho_tw,
                                   int(self.is_source), int(self.ratio_mode), int(dlogits_dtype), int(self.objective),
                                   int(self.global_steps))


def impact_loss_workspace_bytes(B: int, T: int) -> int:
    return load_library().impact_loss_workspace_bytes(B, T)


def impact_loss_workspace_init(workspace: torch.Tensor, stream=None) -> None:
    _check(load_library().impact_loss_workspace_init(workspace.data_ptr(), workspace.numel() * workspace.element_size(),
                                                     _stream(stream)), "impact_loss_workspace_init")


def impact_loss_workspace_status(workspace: torch.Tensor, stream=None) -> int:
    """The workspace's error word (0 = every bounded wait of the loss kernels completed); synchronises."""
    flag = _i32(-1)
    _check(load_library().impact_loss_workspace_status(workspace.data_ptr(), workspace.numel() * workspace.element_size(),
                                                       ctypes.byref(flag), _stream(stream)),
           "impact_loss_workspace_status")
    return flag.value


def new_workspace(B: int, T: int, device="cuda") -> torch.Tensor:
    """Allocates and clears a workspace for batches of B x T steps."""
    ws = torch.empty(impact_loss_workspace_bytes(B, T), dtype=torch.uint8, device=device)
    impact_loss_workspace_init(ws)
    return ws


_TORCH_DTYPE = {DTYPE_F32: torch.float32, DTYPE_BF16: torch.bfloat16}
_DTYPE_CODE = {torch.float32: DTYPE_F32, torch.bfloat16: DTYPE_BF16}


class PreparedCall:
    """A C call with its arguments marshalled once; `()` re-issues it on the given stream.  `keep` holds whatever
    the marshalled pointers point into (the C structs and every tensor of the call), so that the call can be
    re-issued for as long as it exists."""

    def __init__(self, fn, args, what, keep):
        self._fn, self._args, self._what, self._keep = fn, list(args), what, keep

    def __call__(self, stream=None) -> None:
        self._args[-1] = _stream(stream)
        st = self._fn(*self._args)
        if st != OK:
            _check(st, self._what)

    def on_stream(self, cuda_stream: int) -> None:
        """Same as `()`, for a raw cudaStream_t value (skips the torch stream lookup)."""
        self._args[-1] = cuda_stream
        st = self._fn(*self._args)
        if st != OK:
            _check(st, self._what)


def prepare_loss_fwd_bwd(learner_logits, target_logits, worker_logp, actions, rewards, discounts, values,
                         bootstrap_values, coef: Coefficients, *, loss_terms, dlogits, dvalues,
                         vtarget=None, advantage=None, workspace, target_logits_copy=None) -> PreparedCall:
    lib = load_library()
    B, T, A = learner_logits.shape
    ldt = learner_logits.dtype
    if ldt not in _DTYPE_CODE or dlogits.dtype not in _DTYPE_CODE:
        raise ValueError("logits must be float32 or bfloat16")
    f32, bt = torch.float32, (B, T)
    cs = coef.c_struct(_DTYPE_CODE[dlogits.dtype])
    call = impact_loss_call(
        _dev(learner_logits, ldt, (B, T, A), "learner_logits"), _dev(target_logits, ldt, (B, T, A), "target_logits"),
        _dev(worker_logp, f32, bt, "worker_logp"), _dev(actions, torch.int32, bt, "actions"),
        _dev(rewards, f32, bt, "rewards"), _dev(discounts, f32, bt, "discounts"), _dev(values, f32, bt, "values"),
        _dev(bootstrap_values, f32, (B,), "bootstrap_values"),
        coef.rho_bar, coef.c_bar, coef.clip_eps, _DTYPE_CODE[ldt], cs, A, B, T,
        _dev(loss_terms, f32, (NUM_TERMS,), "loss_terms"), _dev(dlogits, dlogits.dtype, (B, T, A), "dlogits"),
        _dev(dvalues, f32, bt, "dvalues"), _dev(vtarget, f32, bt, "vtarget", True),
        _dev(advantage, f32, bt, "advantage", True),
        _dev(workspace, torch.uint8, workspace.shape, "workspace"), workspace.numel(),
        _dev(target_logits_copy, ldt, (B, T, A), "target_logits_copy", True), None)
    return PreparedCall(lib.impact_loss_fwd_bwd_call, [ctypes.byref(call), 0], "impact_loss_fwd_bwd_call",
                        (call, learner_logits, target_logits, worker_logp, actions, rewards, discounts, values,
                         bootstrap_values, loss_terms, dlogits, dvalues, vtarget, advantage, workspace,
                         target_logits_copy))


def new_loss_inputs_record(device="cuda") -> torch.Tensor:
    """Device memory for one impact_loss_inputs record (written by ImpactBuffer.device_step, read by the loss call)."""
    return torch.zeros(ctypes.sizeof(impact_loss_inputs) + 8, dtype=torch.uint8, device=device)


def prepare_loss_fwd_bwd_from_record(record: torch.Tensor, B: int, T: int, A: int, logits_dtype: torch.dtype,
                                     coef: Coefficients, *, loss_terms, dlogits, dvalues, vtarget=None,
                                     advantage=None, workspace) -> PreparedCall:
    """The loss call whose inputs are named by a device record (impact_loss_call.inputs_on_device)."""
    lib = load_library()
    if logits_dtype not in _DTYPE_CODE or dlogits.dtype not in _DTYPE_CODE:
        raise ValueError("logits must be float32 or bfloat16")
    if not record.is_cuda or record.numel() * record.element_size() < ctypes.sizeof(impact_loss_inputs):
        raise ValueError("record: device memory of at least sizeof(impact_loss_inputs) bytes")
    f32, bt = torch.float32, (B, T)
    cs = coef.c_struct(_DTYPE_CODE[dlogits.dtype])
    call = impact_loss_call(
        None, None, None, None, None, None, None, None,
        coef.rho_bar, coef.c_bar, coef.clip_eps, _DTYPE_CODE[logits_dtype], cs, A, B, T,
        _dev(loss_terms, f32, (NUM_TERMS,), "loss_terms"), _dev(dlogits, dlogits.dtype, (B, T, A), "dlogits"),
        _dev(dvalues, f32, bt, "dvalues"), _dev(vtarget, f32, bt, "vtarget", True),
        _dev(advantage, f32, bt, "advantage", True),
        _dev(workspace, torch.uint8, workspace.shape, "workspace"), workspace.numel(), None, record.data_ptr())
    return PreparedCall(lib.impact_loss_fwd_bwd_call, [ctypes.byref(call), 0], "impact_loss_fwd_bwd_call",
                        (call, record, loss_terms, dlogits, dvalues, vtarget, advantage, workspace))


def impact_loss_fwd_bwd(learner_logits, target_logits, worker_logp, actions, rewards, discounts, values,
                        bootstrap_values, coef: Coefficients, *, loss_terms, dlogits, dvalues,
                        vtarget=None, advantage=None, workspace, target_logits_copy=None, stream=None) -> None:
    """Enqueues the categorical IMPACT loss + gradients on `stream` (see include/impact.h)."""
    prepare_loss_fwd_bwd(learner_logits, target_logits, worker_logp, actions, rewards, discounts, values,
                         bootstrap_values, coef, loss_terms=loss_terms, dlogits=dlogits, dvalues=dvalues,
                         vtarget=vtarget, advantage=advantage, workspace=workspace,
                         target_logits_copy=target_logits_copy)(stream)


def impact_loss_fwd_bwd_static_scratch(learner_logits, target_logits, worker_logp, actions, rewards, discounts,
                                       values, bootstrap_values, coef: Coefficients, *, loss_terms, dlogits,
                                       dvalues, vtarget=None, advantage=None, stream=None) -> None:
    """impact_loss_fwd_bwd without a workspace argument, for callers that may not allocate.

    The scratch the kernel needs sits in an array inside the library, so this call takes only
    inputs and outputs.  Batches are limited to 1024 tiles of 128 steps and A <= 64; all calls
    on a device share the array, so keep them ordered on one stream (see include/impact.h).
    """
    lib = load_library()
    B, T, A = learner_logits.shape
    ldt = learner_logits.dtype
    if ldt not in _DTYPE_CODE or dlogits.dtype not in _DTYPE_CODE:
        raise ValueError("logits must be float32 or bfloat16")
    f32, bt = torch.float32, (B, T)
    cs = coef.c_struct(_DTYPE_CODE[dlogits.dtype])
    st = lib.impact_loss_fwd_bwd_static_scratch(
        _dev(learner_logits, ldt, (B, T, A), "learner_logits"), _dev(target_logits, ldt, (B, T, A), "target_logits"),
        _dev(worker_logp, f32, bt, "worker_logp"), _dev(actions, torch.int32, bt, "actions"),
        _dev(rewards, f32, bt, "rewards"), _dev(discounts, f32, bt, "discounts"), _dev(values, f32, bt, "values"),
        _dev(bootstrap_values, f32, (B,), "bootstrap_values"),
        coef.rho_bar, coef.c_bar, coef.clip_eps, ctypes.pointer(cs), B, T, A, _DTYPE_CODE[ldt],
        _dev(loss_terms, f32, (NUM_TERMS,), "loss_terms"), _dev(dlogits, dlogits.dtype, (B, T, A), "dlogits"),
        _dev(dvalues, f32, bt, "dvalues"), _dev(vtarget, f32, bt, "vtarget", True),
        _dev(advantage, f32, bt, "advantage", True), _stream(stream))
    _check(st, "impact_loss_fwd_bwd_static_scratch")


def impact_loss_static_scratch_status(clear: bool = False, stream=None) -> int:
    """Error word of the built-in scratch on the current device (0 = every bounded wait completed); synchronises."""
    flag = _i32(-1)
    _check(load_library().impact_loss_static_scratch_status(ctypes.byref(flag), 1 if clear else 0, _stream(stream)),
           "impact_loss_static_scratch_status")
    return flag.value


def prepare_loss_fwd_bwd_gaussian(learner_mean, learner_logstd, target_mean, target_logstd, worker_logp, actions,
                                  rewards, discounts, values, bootstrap_values, coef: Coefficients, *,
                                  loss_terms, dmean, dlogstd, dvalues, vtarget=None, advantage=None,
                                  workspace) -> PreparedCall:
    lib = load_library()
    B, T, D = learner_mean.shape
    f32, bt, btd = torch.float32, (B, T), (B, T, D)
    cs = coef.c_struct(DTYPE_F32)
    args = [
        _dev(learner_mean, f32, btd, "learner_mean"), _dev(learner_logstd, f32, btd, "learner_logstd"),
        _dev(target_mean, f32, btd, "target_mean"), _dev(target_logstd, f32, btd, "target_logstd"),
        _dev(worker_logp, f32, bt, "worker_logp"), _dev(actions, f32, btd, "actions"),
        _dev(rewards, f32, bt, "rewards"), _dev(discounts, f32, bt, "discounts"), _dev(values, f32, bt, "values"),
        _dev(bootstrap_values, f32, (B,), "bootstrap_values"),
        coef.rho_bar, coef.c_bar, coef.clip_eps, ctypes.pointer(cs), B, T, D,
        _dev(loss_terms, f32, (NUM_TERMS,), "loss_terms"), _dev(dmean, f32, btd, "dmean"),
        _dev(dlogstd, f32, btd, "dlogstd"), _dev(dvalues, f32, bt, "dvalues"),
        _dev(vtarget, f32, bt, "vtarget", True), _dev(advantage, f32, bt, "advantage", True),
        _dev(workspace, torch.uint8, workspace.shape, "workspace"), workspace.numel(), 0,
    ]
    return PreparedCall(lib.impact_loss_fwd_bwd_gaussian, args, "impact_loss_fwd_bwd_gaussian",
                        (cs, learner_mean, learner_logstd, target_mean, target_logstd, worker_logp, actions, rewards,
                         discounts, values, bootstrap_values, loss_terms, dmean, dlogstd, dvalues, vtarget, advantage,
                         workspace))


def impact_loss_fwd_bwd_gaussian(learner_mean, learner_logstd, target_mean, target_logstd, worker_logp, actions,
                                 rewards, discounts, values, bootstrap_values, coef: Coefficients, *,
                                 loss_terms, dmean, dlogstd, dvalues, vtarget=None, advantage=None,
                                 workspace, stream=None) -> None:
    """Enqueues the diagonal-Gaussian IMPACT loss + gradients on `stream`."""
    prepare_loss_fwd_bwd_gaussian(learner_mean, learner_logstd, target_mean, target_logstd, worker_logp, actions,
                                  rewards, discounts, values, bootstrap_values, coef, loss_terms=loss_terms,
                                  dmean=dmean, dlogstd=dlogstd, dvalues=dvalues, vtarget=vtarget,
                                  advantage=advantage, workspace=workspace)(stream)


def impact_gather_rows(src: torch.Tensor, idx: torch.Tensor, dst: torch.Tensor, stream=None) -> None:
    """dst[i] = src[idx[i]] along dim 0, byte-exact; src/dst are dense CUDA tensors of equal row size."""
    if not (src.is_cuda and dst.is_cuda and idx.is_cuda) or idx.dtype != torch.int32:
        raise ValueError("impact_gather_rows needs CUDA tensors and int32 indices")
    if not (src.is_contiguous() and dst.is_contiguous() and idx.is_contiguous()):
        raise ValueError("impact_gather_rows needs dense tensors")
    n = idx.numel()
    row_bytes = (src.numel() // max(src.shape[0], 1)) * src.element_size()
    if dst.shape[0] != n or (dst.numel() // max(n, 1)) * dst.element_size() != row_bytes:
        raise ValueError("dst must hold one source row per index")
    _check(load_library().impact_gather_rows(src.data_ptr(), idx.data_ptr(), n, src.shape[0], row_bytes,
                                             dst.data_ptr(), _stream(stream)), "impact_gather_rows")


def prepare_stream_copy(src: torch.Tensor, read_bytes: int, dst: torch.Tensor, write_bytes: int) -> PreparedCall:
    """impact_stream_copy with its arguments marshalled once (a measurement aid: see include/impact.h)."""
    if not (src.is_cuda and dst.is_cuda and src.is_contiguous() and dst.is_contiguous()):
        raise ValueError("impact_stream_copy needs dense CUDA tensors")
    if src.numel() * src.element_size() < read_bytes or dst.numel() * dst.element_size() < write_bytes:
        raise ValueError("buffers smaller than the byte counts")
    return PreparedCall(load_library().impact_stream_copy, [src.data_ptr(), read_bytes, dst.data_ptr(), write_bytes, 0],
                        "impact_stream_copy", (src, dst))


class ImpactBuffer:
    """Handle of the circular buffer C(N, K); methods are the impact_buffer_* calls."""

    def __init__(self, N: int, K: int, field_bytes, seed: int = 0, sample_mode: int = SAMPLE_UNIFORM,
                 storage: torch.Tensor | None = None, library_owned_storage: bool = False):
        self._lib = load_library()
        self.N, self.K = N, K
        self.field_bytes = [int(b) for b in field_bytes]
        self.n_fields = len(self.field_bytes)
        self._fb = (_sz * self.n_fields)(*self.field_bytes)
        if storage is None and not library_owned_storage:
            # torch owns the ring's device memory, so that slots can be viewed as tensors
            storage = torch.empty(self.storage_bytes(N, self.field_bytes), dtype=torch.uint8, device="cuda")
        self._storage = storage
        h = _vp()
        st = self._lib.impact_buffer_create(N, K, self.n_fields, self._fb, seed, sample_mode,
                                            storage.data_ptr() if storage is not None else None, ctypes.byref(h))
        _check(st, "impact_buffer_create")
        self._h = h
        self._slot = _i32(-1)
        self._k = _i32(-1)

    @staticmethod
    def storage_bytes(N: int, field_bytes) -> int:
        fb = (_sz * len(field_bytes))(*[int(b) for b in field_bytes])
        return load_library().impact_buffer_storage_bytes(N, len(field_bytes), fb)

    def _ptr_array(self, tensors):
        if len(tensors) != self.n_fields:
            raise ValueError("one entry per field expected")
        arr = (_vp * self.n_fields)()
        for f, t in enumerate(tensors):
            if t is None:
                arr[f] = None
                continue
            nbytes = t.numel() * t.element_size()
            if nbytes != self.field_bytes[f] or not t.is_contiguous():
                raise ValueError(f"field {f}: expected {self.field_bytes[f]} dense bytes, got {nbytes}")
            arr[f] = t.data_ptr()
        return arr

    def push(self, fields, stream=None) -> int | None:
        """impact_buffer_push: returns the slot, or None when the buffer is full."""
        host = [t.is_cuda for t in fields if t is not None]
        if any(host) and not all(host):
            raise ValueError("push sources must be all on the device or all on the host")
        loc = SRC_DEVICE if (not host or host[0]) else SRC_HOST
        st = self._lib.impact_buffer_push(self._h, self._ptr_array(fields), loc, ctypes.byref(self._slot),
                                          _stream(stream))
        if _check(st, "impact_buffer_push", allow=(ERR_FULL,)) == ERR_FULL:
            return None
        return self._slot.value

    def sample(self, gather_dst=None, stream=None):
        """impact_buffer_sample: returns (slot, k_before), or None when the buffer is empty."""
        arr = None
        if gather_dst is not None:
            if not all(t is None or t.is_cuda for t in gather_dst):
                raise ValueError("gather destinations must be CUDA tensors")
            arr = self._ptr_array(gather_dst)
        st = self._lib.impact_buffer_sample(self._h, ctypes.byref(self._slot), ctypes.byref(self._k), arr,
                                            _stream(stream))
        if _check(st, "impact_buffer_sample", allow=(ERR_EMPTY,)) == ERR_EMPTY:
            return None
        return self._slot.value, self._k.value

    def append(self, slot: int, field: int, src: torch.Tensor, stream=None) -> None:
        if not src.is_cuda or not src.is_contiguous() or src.numel() * src.element_size() != self.field_bytes[field]:
            raise ValueError("append source must be a dense CUDA tensor of the field's size")
        _check(self._lib.impact_buffer_append(self._h, slot, field, src.data_ptr(), _stream(stream)),
               "impact_buffer_append")

    def slot_ptr(self, slot: int, field: int) -> int:
        p = self._lib.impact_buffer_slot_ptr(self._h, slot, field)
        if not p:
            raise ValueError("bad slot or field")
        return p

    def slot_view(self, slot: int, field: int, dtype: torch.dtype, shape) -> torch.Tensor:
        """Zero-copy tensor over one field of a slot (needs torch-owned storage)."""
        if self._storage is None:
            raise ValueError("slot_view needs torch-owned storage")
        off = self.slot_ptr(slot, field) - self._storage.data_ptr()
        n = self.field_bytes[field]
        return self._storage[off:off + n].view(dtype).view(*shape)

    def live(self) -> int:
        return _check(self._lib.impact_buffer_live(self._h), "impact_buffer_live", allow=tuple(range(1, self.N + 1)))

    def export_state(self) -> bytes:
        n = self._lib.impact_buffer_state_bytes(self._h)
        buf = ctypes.create_string_buffer(n)
        _check(self._lib.impact_buffer_export_state(self._h, buf, n), "impact_buffer_export_state")
        return buf.raw

    def import_state(self, blob: bytes) -> None:
        _check(self._lib.impact_buffer_import_state(self._h, blob, len(blob)), "impact_buffer_import_state")

    # ---- bookkeeping on the device -------------------------------------------------------------------------
    def device_begin(self, stream=None) -> None:
        _check(self._lib.impact_buffer_device_begin(self._h, _stream(stream)), "impact_buffer_device_begin")

    def device_end(self, stream=None) -> None:
        _check(self._lib.impact_buffer_device_end(self._h, _stream(stream)), "impact_buffer_device_end")

    def prepare_device_step(self, field_map=None, learner_logits=None, values=None, bootstrap_values=None,
                            push_sources: torch.Tensor | None = None, record: torch.Tensor | None = None) -> PreparedCall:
        """impact_buffer_device_step with its arguments marshalled once.  field_map: dict name -> ring field index
        (missing = not in the ring); push_sources: int64 CUDA tensor [n_candidates, n_fields + 1] of device addresses
        (0 = none); record: from new_loss_inputs_record()."""
        fm = None
        if record is not None:
            m = field_map or {}
            fm = impact_ring_field_map(*[int(m.get(n, -1)) for n in ("actions", "rewards", "discounts", "worker_logp",
                                                                      "target_logits")])
        ncand = 0
        if push_sources is not None:
            if not push_sources.is_cuda or push_sources.dtype != torch.int64 or push_sources.dim() != 2 or \
                    push_sources.shape[1] != self.n_fields + 1 or not push_sources.is_contiguous():
                raise ValueError("push_sources: contiguous int64 CUDA tensor [n_candidates, n_fields + 1]")
            ncand = push_sources.shape[0]
        ptr = lambda t: None if t is None else t.data_ptr()
        args = [self._h, ctypes.byref(fm) if fm is not None else None, ptr(learner_logits), ptr(values),
                ptr(bootstrap_values), ptr(push_sources), ncand, ptr(record), 0]
        return PreparedCall(self._lib.impact_buffer_device_step, args, "impact_buffer_device_step",
                            (fm, learner_logits, values, bootstrap_values, push_sources, record))

    def device_events(self, max_events: int = 4096, stream=None):
        """The most recent (op, status, slot, k_before) outcomes, oldest first (op 1 = push, 2 = sample)."""
        buf = (_i32 * (4 * max_events))()
        n = _i32(0)
        _check(self._lib.impact_buffer_device_events(self._h, buf, max_events, ctypes.byref(n), _stream(stream)),
               "impact_buffer_device_events")
        return [tuple(buf[4 * i:4 * i + 4]) for i in range(n.value)]

    def close(self) -> None:
        if self._h:
            self._lib.impact_buffer_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

"""ctypes binding of liblite3r.so: argument marshalling only, every step runs in the CUDA kernels.

The functions carry the C names (``lite3r_quantize_fp8``, ``lite3r_sla_plan``, ``lite3r_sla_forward``);
torch is used for device memory and streams.  There is no fallback: if the shared library is missing
the import of any compute function raises.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "liblite3r.so")
_lib = None

F32, BF16, F16 = 0, 1, 2
OUT_DTYPES = {torch.float32: F32, torch.bfloat16: BF16, torch.float16: F16}
PHI_SOFTMAX, PHI_ELU1 = 0, 1
PHI_CODES = {"softmax": PHI_SOFTMAX, "elu1": PHI_ELU1}


class Lite3rError(RuntimeError):
    pass


class Shape(C.Structure):
    _fields_ = [("batch", C.c_int), ("heads", C.c_int), ("tokens", C.c_int), ("head_dim", C.c_int), ("block", C.c_int)]


class Tensor(C.Structure):
    _fields_ = [("ptr", C.c_void_p), ("dtype", C.c_int), ("stride_b", C.c_longlong), ("stride_h", C.c_longlong),
                ("stride_n", C.c_longlong)]


class Fp8(C.Structure):
    _fields_ = [("codes", C.c_void_p), ("scales", C.c_void_p), ("colsum", C.c_void_p)]


class Plan(C.Structure):
    _fields_ = [("cls", C.c_void_p), ("crit_idx", C.c_void_p), ("marg_idx", C.c_void_p), ("k_crit", C.c_int),
                ("k_marg", C.c_int), ("k_neg", C.c_int)]


EXPORTS = ("lite3r_fp8_sizes", "lite3r_plan_sizes", "lite3r_forward_workspace", "lite3r_quantize_fp8",
           "lite3r_sla_plan", "lite3r_sla_forward", "lite3r_status_string", "lite3r_last_cuda_error",
           "lite3r_launch_count", "lite3r_profile_enable", "lite3r_profile_stage_ms",
           "lite3r_sla_forward_static_scratch", "lite3r_quantize_fp8_qkv", "lite3r_selftest_wait_expiry",
           "lite3r_sla_forward_begin", "lite3r_sla_forward_finish", "lite3r_forward_workspace_planned",
           "lite3r_workspace_layout", "lite3r_quantize_rows_fp8", "lite3r_linear_fp8", "lite3r_qkv_project_fp8",
           "lite3r_train_workspace", "lite3r_sla_linear_branch", "lite3r_mse_distill", "lite3r_proj_lin_backward",
           "lite3r_plan_variant", "lite3r_attention_plain_stores")
STATIC_SCRATCH_BYTES = 32 << 20  # LITE3R_STATIC_SCRATCH_BYTES


def lib() -> C.CDLL:
    """Loads the shared library once; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise Lite3rError(f"{_LIB_PATH} is missing: build it with `python -m paper_2605_11354_b200.build`")
    L = C.CDLL(_LIB_PATH)
    sz = C.POINTER(C.c_size_t)
    ip = C.POINTER(C.c_int)
    L.lite3r_fp8_sizes.argtypes = [C.POINTER(Shape), sz, sz, sz]
    L.lite3r_plan_sizes.argtypes = [C.POINTER(Shape), C.c_double, C.c_double, sz, sz, sz, ip, ip, ip]
    L.lite3r_forward_workspace.argtypes = [C.POINTER(Shape), C.c_double, C.c_double, sz]
    L.lite3r_quantize_fp8.argtypes = [C.POINTER(Tensor), C.POINTER(Shape), Fp8, C.c_void_p]
    L.lite3r_quantize_fp8_qkv.argtypes = [C.POINTER(Tensor), C.POINTER(Tensor), C.POINTER(Tensor), C.POINTER(Shape), Fp8,
                                          Fp8, Fp8, C.c_void_p]
    L.lite3r_quantize_fp8_qkv.restype = C.c_int
    L.lite3r_sla_plan.argtypes = [C.POINTER(Fp8), C.POINTER(Fp8), C.POINTER(Shape), C.c_double, C.c_double,
                                  C.POINTER(Plan), C.c_void_p]
    L.lite3r_forward_workspace_planned.argtypes = [C.POINTER(Shape), C.c_double, C.c_double, sz]
    L.lite3r_forward_workspace_planned.restype = C.c_int
    L.lite3r_workspace_layout.argtypes = [C.POINTER(Shape), C.c_double, C.c_double, C.c_int, sz]
    L.lite3r_workspace_layout.restype = C.c_int
    L.lite3r_sla_forward.argtypes = [C.POINTER(Fp8), C.POINTER(Fp8), C.POINTER(Fp8), C.c_void_p, C.c_longlong,
                                     C.POINTER(Shape), C.c_double, C.c_double, C.c_int, C.POINTER(Plan), C.c_void_p,
                                     C.c_int, C.c_longlong, C.c_longlong, C.c_longlong, C.c_void_p, C.c_size_t,
                                     C.c_void_p, C.c_void_p]
    L.lite3r_sla_forward_static_scratch.argtypes = [C.POINTER(Fp8), C.POINTER(Fp8), C.POINTER(Fp8), C.c_void_p,
                                                    C.c_longlong, C.POINTER(Shape), C.c_int, C.POINTER(Plan),
                                                    C.c_void_p, C.c_int, C.c_longlong, C.c_longlong, C.c_longlong,
                                                    C.c_void_p, C.c_void_p]
    L.lite3r_sla_forward_static_scratch.restype = C.c_int
    L.lite3r_sla_forward_begin.argtypes = [C.POINTER(Fp8), C.POINTER(Fp8), C.c_void_p, C.c_longlong, C.POINTER(Shape),
                                           C.c_int, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_size_t, C.c_void_p,
                                           C.c_void_p]
    L.lite3r_sla_forward_begin.restype = C.c_int
    L.lite3r_sla_forward_finish.argtypes = [C.POINTER(Fp8), C.POINTER(Fp8), C.POINTER(Fp8), C.POINTER(Shape), C.c_int,
                                            C.POINTER(Plan), C.c_void_p, C.c_int, C.c_longlong, C.c_longlong,
                                            C.c_longlong, C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
    L.lite3r_sla_forward_finish.restype = C.c_int
    L.lite3r_quantize_rows_fp8.argtypes = [C.c_void_p, C.c_int, C.c_longlong, C.c_int, C.c_int, C.c_void_p, C.c_void_p,
                                           C.c_void_p]
    L.lite3r_quantize_rows_fp8.restype = C.c_int
    L.lite3r_linear_fp8.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int,
                                    C.c_void_p, C.c_int, C.c_longlong, C.c_void_p, C.c_void_p]
    L.lite3r_linear_fp8.restype = C.c_int
    L.lite3r_qkv_project_fp8.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(Shape),
                                         C.c_int, Fp8, Fp8, Fp8, C.c_void_p, C.c_void_p]
    L.lite3r_qkv_project_fp8.restype = C.c_int
    L.lite3r_train_workspace.argtypes = [C.POINTER(Shape), C.c_double, C.c_double, sz]
    L.lite3r_train_workspace.restype = C.c_int
    L.lite3r_sla_linear_branch.argtypes = [C.POINTER(Fp8), C.POINTER(Fp8), C.POINTER(Fp8), C.POINTER(Shape), C.c_int,
                                           C.POINTER(Plan), C.c_void_p, C.c_int, C.c_longlong, C.c_longlong,
                                           C.c_longlong, C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
    L.lite3r_sla_linear_branch.restype = C.c_int
    L.lite3r_mse_distill.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_longlong, C.c_void_p, C.c_void_p, C.c_void_p,
                                     C.c_size_t, C.c_void_p]
    L.lite3r_mse_distill.restype = C.c_int
    L.lite3r_proj_lin_backward.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(Shape), C.c_void_p, C.c_void_p, C.c_size_t,
                                           C.c_void_p, C.c_void_p]
    L.lite3r_proj_lin_backward.restype = C.c_int
    L.lite3r_selftest_wait_expiry.argtypes = [C.c_void_p, C.c_ulonglong, C.c_void_p]
    L.lite3r_selftest_wait_expiry.restype = C.c_int
    L.lite3r_status_string.argtypes = [C.c_int]
    L.lite3r_status_string.restype = C.c_char_p
    L.lite3r_last_cuda_error.restype = C.c_int
    L.lite3r_launch_count.restype = C.c_longlong
    L.lite3r_plan_variant.argtypes = [C.c_int]
    L.lite3r_plan_variant.restype = C.c_int
    L.lite3r_attention_plain_stores.argtypes = [C.c_int]
    L.lite3r_attention_plain_stores.restype = C.c_int
    L.lite3r_profile_enable.argtypes = [C.c_int]
    L.lite3r_profile_enable.restype = C.c_int
    L.lite3r_profile_stage_ms.argtypes = [C.POINTER(C.c_float)]
    L.lite3r_profile_stage_ms.restype = C.c_int
    for name in EXPORTS[:6]:
        getattr(L, name).restype = C.c_int
    _lib = L
    return L


def _check(status: int, what: str) -> None:
    if status != 0:
        L = lib()
        msg = L.lite3r_status_string(status).decode()
        extra = f" (cudaError {L.lite3r_last_cuda_error()})" if status == 4 else ""
        raise Lite3rError(f"{what}: {msg}{extra}")


def _stream_ptr(stream) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return int(s.cuda_stream)


def selftest_wait_expiry(status: torch.Tensor, limit_ns: int, stream=None) -> None:
    """Runs the bounded-wait self-test kernel; `status` (CUDA int32 [1]) is non-zero afterwards."""
    _check(lib().lite3r_selftest_wait_expiry(status.data_ptr(), limit_ns, _stream_ptr(stream)),
           "lite3r_selftest_wait_expiry")


def launch_count() -> int:
    return int(lib().lite3r_launch_count())


def lite3r_attention_plain_stores(on: bool) -> None:
    """Test hook: forces the attention kernel's plain-store output path."""
    _check(lib().lite3r_attention_plain_stores(1 if on else 0), "lite3r_attention_plain_stores")


def lite3r_plan_variant(variant: int) -> None:
    """Test hook: forces one of the plan kernels (0 = chosen by size)."""
    _check(lib().lite3r_plan_variant(int(variant)), "lite3r_plan_variant")


def profile_enable(on: bool) -> None:
    _check(lib().lite3r_profile_enable(1 if on else 0), "lite3r_profile_enable")


def profile_stage_ms():
    """(prep, summary, aggregation, attention) milliseconds of the last forward; blocks until it has finished."""
    ms = (C.c_float * 4)()
    _check(lib().lite3r_profile_stage_ms(ms), "lite3r_profile_stage_ms")
    return tuple(float(x) for x in ms)


# ----------------------------------------------------------------------------- size queries (host only)
def lite3r_fp8_sizes(shape: Shape):
    a, b, c = C.c_size_t(), C.c_size_t(), C.c_size_t()
    _check(lib().lite3r_fp8_sizes(C.byref(shape), C.byref(a), C.byref(b), C.byref(c)), "lite3r_fp8_sizes")
    return a.value, b.value, c.value


def lite3r_plan_sizes(shape: Shape, crit: float, neg: float):
    a, b, c = C.c_size_t(), C.c_size_t(), C.c_size_t()
    kc, km, kn = C.c_int(), C.c_int(), C.c_int()
    _check(lib().lite3r_plan_sizes(C.byref(shape), crit, neg, C.byref(a), C.byref(b), C.byref(c), C.byref(kc),
                                   C.byref(km), C.byref(kn)), "lite3r_plan_sizes")
    return a.value, b.value, c.value, kc.value, km.value, kn.value


def lite3r_forward_workspace(shape: Shape, crit: float, neg: float) -> int:
    a = C.c_size_t()
    _check(lib().lite3r_forward_workspace(C.byref(shape), crit, neg, C.byref(a)), "lite3r_forward_workspace")
    return a.value


def lite3r_forward_workspace_planned(shape: Shape, crit: float, neg: float) -> int:
    """Workspace bytes of lite3r_sla_forward called without a plan (the plan is then built inside the workspace)."""
    a = C.c_size_t()
    _check(lib().lite3r_forward_workspace_planned(C.byref(shape), crit, neg, C.byref(a)),
           "lite3r_forward_workspace_planned")
    return a.value


def lite3r_workspace_layout(shape: Shape, crit: float, neg: float, plan_inside: bool = False):
    """Byte offsets of the six parts of the forward's workspace (summaries, aggregates, zeta, fp16 V, classes, lists)."""
    arr = (C.c_size_t * 6)()
    _check(lib().lite3r_workspace_layout(C.byref(shape), crit, neg, 1 if plan_inside else 0, arr),
           "lite3r_workspace_layout")
    return tuple(int(x) for x in arr)


# ----------------------------------------------------------------------------- device buffers
@dataclass
class Fp8Tensor:
    codes: torch.Tensor  # uint8 [B,H,Nb*Bs,D]
    scales: torch.Tensor  # fp32 [B,H,Nb]
    colsum: torch.Tensor | None  # int32 [B,H,Nb,D]; None: the quantiser skips the column sums (only Q and K need them)

    def c_struct(self) -> Fp8:
        return Fp8(self.codes.data_ptr(), self.scales.data_ptr(),
                   self.colsum.data_ptr() if self.colsum is not None else None)


@dataclass
class PlanBuffers:
    cls: torch.Tensor  # int8 [B,H,Nb,Nb]
    crit_idx: torch.Tensor  # int32 [B,H,Nb,k_crit]
    marg_idx: torch.Tensor  # int32 [B,H,Nb,k_marg]
    k_crit: int
    k_marg: int
    k_neg: int

    def c_struct(self) -> Plan:
        return Plan(self.cls.data_ptr(), self.crit_idx.data_ptr() if self.k_crit else None,
                    self.marg_idx.data_ptr() if self.k_marg else None, self.k_crit, self.k_marg, self.k_neg)


def alloc_fp8(shape: Shape, device, colsum: bool = True) -> Fp8Tensor:
    nb = -(-shape.tokens // shape.block)
    B, H, D = shape.batch, shape.heads, shape.head_dim
    return Fp8Tensor(torch.empty((B, H, nb * shape.block, D), dtype=torch.uint8, device=device),
                     torch.empty((B, H, nb), dtype=torch.float32, device=device),
                     torch.empty((B, H, nb, D), dtype=torch.int32, device=device) if colsum else None)


def alloc_plan(shape: Shape, crit: float, neg: float, device) -> PlanBuffers:
    _, _, _, kc, km, kn = lite3r_plan_sizes(shape, crit, neg)
    nb = -(-shape.tokens // shape.block)
    B, H = shape.batch, shape.heads
    return PlanBuffers(torch.empty((B, H, nb, nb), dtype=torch.int8, device=device),
                       torch.empty((B, H, nb, max(kc, 1)), dtype=torch.int32, device=device)[..., :kc],
                       torch.empty((B, H, nb, max(km, 1)), dtype=torch.int32, device=device)[..., :km], kc, km, kn)


# ----------------------------------------------------------------------------- the three calls
def lite3r_quantize_fp8(x: torch.Tensor, shape: Shape, out: Fp8Tensor, stream=None) -> None:
    """x: CUDA tensor [B,H,N,D] (any b/h/n strides, contiguous D), fp32 or bf16."""
    if not x.is_cuda or x.dim() != 4 or x.stride(3) != 1:
        raise Lite3rError("lite3r_quantize_fp8: x must be a CUDA tensor [B,H,N,D] with contiguous D")
    dtype = {torch.float32: F32, torch.bfloat16: BF16}.get(x.dtype)
    if dtype is None:
        raise Lite3rError("lite3r_quantize_fp8: dtype must be float32 or bfloat16")
    t = Tensor(x.data_ptr(), dtype, x.stride(0), x.stride(1), x.stride(2))
    _check(lib().lite3r_quantize_fp8(C.byref(t), C.byref(shape), out.c_struct(), _stream_ptr(stream)),
           "lite3r_quantize_fp8")


def _source(x: torch.Tensor, what: str) -> Tensor:
    if not x.is_cuda or x.dim() != 4 or x.stride(3) != 1:
        raise Lite3rError(f"{what}: sources must be CUDA tensors [B,H,N,D] with contiguous D")
    dtype = {torch.float32: F32, torch.bfloat16: BF16}.get(x.dtype)
    if dtype is None:
        raise Lite3rError(f"{what}: dtype must be float32 or bfloat16")
    return Tensor(x.data_ptr(), dtype, x.stride(0), x.stride(1), x.stride(2))


def lite3r_quantize_fp8_qkv(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, shape: Shape, q_out: Fp8Tensor,
                            k_out: Fp8Tensor, v_out: Fp8Tensor, stream=None) -> None:
    """Q, K and V of one attention call quantised by a single launch (same results as three single calls)."""
    tq, tk, tv = (_source(x, "lite3r_quantize_fp8_qkv") for x in (q, k, v))
    _check(lib().lite3r_quantize_fp8_qkv(C.byref(tq), C.byref(tk), C.byref(tv), C.byref(shape), q_out.c_struct(),
                                         k_out.c_struct(), v_out.c_struct(), _stream_ptr(stream)),
           "lite3r_quantize_fp8_qkv")


def lite3r_sla_plan(q: Fp8Tensor, k: Fp8Tensor, shape: Shape, crit: float, neg: float, plan: PlanBuffers,
                    stream=None) -> None:
    p = plan.c_struct()
    qs, ks = q.c_struct(), k.c_struct()
    _check(lib().lite3r_sla_plan(C.byref(qs), C.byref(ks), C.byref(shape), crit, neg, C.byref(p),
                                 _stream_ptr(stream)), "lite3r_sla_plan")
    assert (p.k_crit, p.k_marg, p.k_neg) == (plan.k_crit, plan.k_marg, plan.k_neg)


def _check_out(out: torch.Tensor, what: str) -> int:
    if out.dtype not in OUT_DTYPES or not out.is_cuda or out.dim() != 4 or out.stride(3) != 1:
        raise Lite3rError(f"{what}: out must be a CUDA float32 / bfloat16 / float16 tensor [B,H,N,D] with contiguous D")
    return OUT_DTYPES[out.dtype]


def lite3r_sla_forward(q: Fp8Tensor, k: Fp8Tensor, v: Fp8Tensor, proj: torch.Tensor, shape: Shape, phi: int,
                       plan, out: torch.Tensor, workspace: torch.Tensor, device_status=None,
                       stream=None, crit: float = 0.0, neg: float = 0.0) -> None:
    """proj: CUDA fp32 [H,D,D] or [D,D] (shared); out: CUDA fp32 / bf16 / fp16 [B,H,N,D] view with contiguous D
    (its dtype selects the output type).  plan=None: the plan is built inside the workspace from crit / neg."""
    if proj.dtype != torch.float32 or not proj.is_cuda or not proj.is_contiguous():
        raise Lite3rError("lite3r_sla_forward: proj must be a contiguous CUDA float32 tensor")
    out_dtype = _check_out(out, "lite3r_sla_forward")
    head_stride = proj.stride(0) if proj.dim() == 3 else 0
    p = plan.c_struct() if plan is not None else None
    qs, ks, vs = q.c_struct(), k.c_struct(), v.c_struct()
    _check(lib().lite3r_sla_forward(C.byref(qs), C.byref(ks), C.byref(vs), proj.data_ptr(), head_stride,
                                    C.byref(shape), crit, neg, phi, C.byref(p) if p is not None else None,
                                    out.data_ptr(), out_dtype, out.stride(0), out.stride(1),
                                    out.stride(2), workspace.data_ptr(), workspace.numel() * workspace.element_size(),
                                    device_status.data_ptr() if device_status is not None else None,
                                    _stream_ptr(stream)), "lite3r_sla_forward")


def lite3r_sla_forward_begin(k: Fp8Tensor, v: Fp8Tensor, proj: torch.Tensor, shape: Shape, phi: int,
                             plan: PlanBuffers, workspace: torch.Tensor, device_status=None, stream=None) -> None:
    """First half of the forward (summaries, fp16 V): needs only the plan's class counts, not its contents."""
    if proj.dtype != torch.float32 or not proj.is_cuda or not proj.is_contiguous():
        raise Lite3rError("lite3r_sla_forward_begin: proj must be a contiguous CUDA float32 tensor")
    head_stride = proj.stride(0) if proj.dim() == 3 else 0
    ks, vs = k.c_struct(), v.c_struct()
    _check(lib().lite3r_sla_forward_begin(C.byref(ks), C.byref(vs), proj.data_ptr(), head_stride, C.byref(shape), phi,
                                          plan.k_crit, plan.k_marg, plan.k_neg, workspace.data_ptr(),
                                          workspace.numel() * workspace.element_size(),
                                          device_status.data_ptr() if device_status is not None else None,
                                          _stream_ptr(stream)), "lite3r_sla_forward_begin")


def lite3r_sla_forward_finish(q: Fp8Tensor, k: Fp8Tensor, v: Fp8Tensor, shape: Shape, phi: int, plan: PlanBuffers,
                              out: torch.Tensor, workspace: torch.Tensor, device_status=None, stream=None) -> None:
    """Second half of the forward (aggregation, attention, linear output, sum); after begin and the plan."""
    out_dtype = _check_out(out, "lite3r_sla_forward_finish")
    p = plan.c_struct()
    qs, ks, vs = q.c_struct(), k.c_struct(), v.c_struct()
    _check(lib().lite3r_sla_forward_finish(C.byref(qs), C.byref(ks), C.byref(vs), C.byref(shape), phi, C.byref(p),
                                           out.data_ptr(), out_dtype, out.stride(0), out.stride(1), out.stride(2),
                                           workspace.data_ptr(), workspace.numel() * workspace.element_size(),
                                           device_status.data_ptr() if device_status is not None else None,
                                           _stream_ptr(stream)), "lite3r_sla_forward_finish")


def lite3r_sla_forward_static_scratch(q: Fp8Tensor, k: Fp8Tensor, v: Fp8Tensor, proj: torch.Tensor, shape: Shape,
                                      phi: int, plan: PlanBuffers, out: torch.Tensor, device_status=None,
                                      stream=None) -> None:
    """lite3r_sla_forward for callers that may not allocate: the scratch is a fixed 32 MiB array inside the
    library, so no workspace is passed.  The first call on a device is the one that makes CUDA load the array (32 MiB
    of device memory are taken then): make it at start-up; later calls allocate nothing.  Raises "workspace too small"
    when the shape needs more than the array holds.  Calls on one device share the array: do not let two of them
    overlap on the GPU."""
    if proj.dtype != torch.float32 or not proj.is_cuda or not proj.is_contiguous():
        raise Lite3rError("lite3r_sla_forward_static_scratch: proj must be a contiguous CUDA float32 tensor")
    out_dtype = _check_out(out, "lite3r_sla_forward_static_scratch")
    head_stride = proj.stride(0) if proj.dim() == 3 else 0
    p = plan.c_struct()
    qs, ks, vs = q.c_struct(), k.c_struct(), v.c_struct()
    _check(lib().lite3r_sla_forward_static_scratch(
        C.byref(qs), C.byref(ks), C.byref(vs), proj.data_ptr(), head_stride, C.byref(shape), phi, C.byref(p),
        out.data_ptr(), out_dtype, out.stride(0), out.stride(1), out.stride(2),
        device_status.data_ptr() if device_status is not None else None, _stream_ptr(stream)),
        "lite3r_sla_forward_static_scratch")


# ----------------------------------------------------------------------------- FP8 linear layer in front of the attention
def lite3r_quantize_rows_fp8(x: torch.Tensor, stream=None):
    """Per-row scaled e4m3 quantisation of a CUDA matrix [rows, cols] (fp32 or bf16, contiguous columns):
    per token for activations, per output row for weights.  Returns (codes uint8 [rows, cols], scales fp32 [rows])."""
    if not x.is_cuda or x.dim() != 2 or x.stride(1) != 1:
        raise Lite3rError("lite3r_quantize_rows_fp8: x must be a CUDA matrix with contiguous columns")
    dtype = {torch.float32: F32, torch.bfloat16: BF16}.get(x.dtype)
    if dtype is None:
        raise Lite3rError("lite3r_quantize_rows_fp8: dtype must be float32 or bfloat16")
    codes = torch.empty(x.shape, dtype=torch.uint8, device=x.device)
    scales = torch.empty(x.shape[0], dtype=torch.float32, device=x.device)
    _check(lib().lite3r_quantize_rows_fp8(x.data_ptr(), dtype, x.stride(0), x.shape[0], x.shape[1], codes.data_ptr(),
                                          scales.data_ptr(), _stream_ptr(stream)), "lite3r_quantize_rows_fp8")
    return codes, scales


def lite3r_linear_fp8(x_codes, x_scales, w_codes, w_scales, bias, y: torch.Tensor, device_status=None, stream=None):
    """y = x_q W_q^T + b on e4m3 operands ([rows, d_in] x [d_out, d_in]); y: CUDA [rows, d_out] fp32 / bf16 / fp16."""
    if y.dtype not in OUT_DTYPES or not y.is_cuda or y.dim() != 2 or y.stride(1) != 1:
        raise Lite3rError("lite3r_linear_fp8: y must be a CUDA float32 / bfloat16 / float16 matrix")
    rows, d_in = x_codes.shape
    d_out = w_codes.shape[0]
    _check(lib().lite3r_linear_fp8(x_codes.data_ptr(), x_scales.data_ptr(), w_codes.data_ptr(), w_scales.data_ptr(),
                                   bias.data_ptr() if bias is not None else None, rows, d_in, d_out, y.data_ptr(),
                                   OUT_DTYPES[y.dtype], y.stride(0),
                                   device_status.data_ptr() if device_status is not None else None,
                                   _stream_ptr(stream)), "lite3r_linear_fp8")


def lite3r_qkv_project_fp8(x_codes, x_scales, w_codes, w_scales, bias, shape: Shape, q_out: Fp8Tensor, k_out: Fp8Tensor,
                           v_out: Fp8Tensor, device_status=None, stream=None):
    """qkv projection on e4m3 operands with the block quantiser fused into its epilogue: fills the three Fp8Tensors
    the attention calls take.  x_codes [B*N, d_model], w_codes [3*H*64, d_model] ordered (q | k | v) x head x 64."""
    _check(lib().lite3r_qkv_project_fp8(x_codes.data_ptr(), x_scales.data_ptr(), w_codes.data_ptr(), w_scales.data_ptr(),
                                        bias.data_ptr() if bias is not None else None, C.byref(shape),
                                        x_codes.shape[1], q_out.c_struct(), k_out.c_struct(), v_out.c_struct(),
                                        device_status.data_ptr() if device_status is not None else None,
                                        _stream_ptr(stream)), "lite3r_qkv_project_fp8")


# ----------------------------------------------------------------------------- training side of the projection
def lite3r_train_workspace(shape: Shape, crit: float, neg: float) -> int:
    a = C.c_size_t()
    _check(lib().lite3r_train_workspace(C.byref(shape), crit, neg, C.byref(a)), "lite3r_train_workspace")
    return a.value


def lite3r_sla_linear_branch(q: Fp8Tensor, k: Fp8Tensor, v: Fp8Tensor, shape: Shape, phi: int, plan: PlanBuffers,
                             out: torch.Tensor, workspace: torch.Tensor, device_status=None, stream=None) -> None:
    """O_lin (the linear branch before the projection) into `out` (CUDA fp32 / bf16 / fp16 [B,H,N,D])."""
    out_dtype = _check_out(out, "lite3r_sla_linear_branch")
    p = plan.c_struct()
    qs, ks, vs = q.c_struct(), k.c_struct(), v.c_struct()
    _check(lib().lite3r_sla_linear_branch(C.byref(qs), C.byref(ks), C.byref(vs), C.byref(shape), phi, C.byref(p),
                                          out.data_ptr(), out_dtype, out.stride(0), out.stride(1), out.stride(2),
                                          workspace.data_ptr(), workspace.numel() * workspace.element_size(),
                                          device_status.data_ptr() if device_status is not None else None,
                                          _stream_ptr(stream)), "lite3r_sla_linear_branch")


def lite3r_mse_distill(student: torch.Tensor, teacher: torch.Tensor, grad, loss: torch.Tensor, workspace: torch.Tensor,
                       stream=None) -> None:
    """loss (CUDA float64 [1]) = MSE(student, teacher); grad (CUDA bf16, same shape, or None) = its gradient."""
    if student.dtype != teacher.dtype or student.dtype not in (torch.float32, torch.bfloat16):
        raise Lite3rError("lite3r_mse_distill: student and teacher must both be float32 or bfloat16")
    if not (student.is_contiguous() and teacher.is_contiguous()) or student.shape != teacher.shape:
        raise Lite3rError("lite3r_mse_distill: contiguous tensors of one shape")
    _check(lib().lite3r_mse_distill(student.data_ptr(), teacher.data_ptr(), OUT_DTYPES[student.dtype], student.numel(),
                                    grad.data_ptr() if grad is not None else None, loss.data_ptr(), workspace.data_ptr(),
                                    workspace.numel() * workspace.element_size(), _stream_ptr(stream)),
           "lite3r_mse_distill")


def lite3r_proj_lin_backward(o_lin: torch.Tensor, d_out: torch.Tensor, shape: Shape, d_proj: torch.Tensor,
                             workspace: torch.Tensor, device_status=None, stream=None) -> None:
    """d_proj (CUDA fp32 [H,64,64]) = sum over batch and tokens of o_lin^T d_out (both CUDA bf16 contiguous [B,H,N,64])."""
    for t in (o_lin, d_out):
        if t.dtype != torch.bfloat16 or not t.is_contiguous():
            raise Lite3rError("lite3r_proj_lin_backward: o_lin and d_out must be contiguous bfloat16")
    _check(lib().lite3r_proj_lin_backward(o_lin.data_ptr(), d_out.data_ptr(), C.byref(shape), d_proj.data_ptr(),
                                          workspace.data_ptr(), workspace.numel() * workspace.element_size(),
                                          device_status.data_ptr() if device_status is not None else None,
                                          _stream_ptr(stream)), "lite3r_proj_lin_backward")


# ----------------------------------------------------------------------------- whole path
class SlaForward:
    """Pre-allocated buffers for one shape; ``run`` enqueues quantise x3 + plan + forward and returns ``out``."""

    def __init__(self, batch, heads, tokens, block, crit, neg, phi="softmax", device="cuda:0", head_dim=64,
                 out_dtype=torch.float32, plan_inside=False):
        """out_dtype: dtype of the engine's own output tensor.  plan_inside: let lite3r_sla_forward build the block
        plan inside its workspace (plan=NULL) instead of calling lite3r_sla_plan."""
        self.shape = Shape(batch, heads, tokens, head_dim, block)
        self.plan_inside = bool(plan_inside)
        self.crit, self.neg, self.phi = float(crit), float(neg), PHI_CODES[phi]
        self.device = torch.device(device)
        self.q8, self.k8 = (alloc_fp8(self.shape, self.device) for _ in range(2))
        self.v8 = alloc_fp8(self.shape, self.device, colsum=False)  # the block plan pools Q and K only
        self.plan = alloc_plan(self.shape, self.crit, self.neg, self.device)
        nbytes = (lite3r_forward_workspace_planned if self.plan_inside else lite3r_forward_workspace)(
            self.shape, self.crit, self.neg)
        self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
        off = (-self.workspace.data_ptr()) % 256
        self.workspace = self.workspace[off:off + nbytes]
        self.out = torch.empty((batch, heads, tokens, head_dim), dtype=out_dtype, device=self.device)
        self.status = torch.zeros(1, dtype=torch.int32, device=self.device)
        self._side = None  # stream of the overlapped first half of the forward, made on first use
        self._graph = None  # (CUDA graph of one whole step, key of the tensors it was captured on)

    def quantize(self, q, k, v, stream=None):
        if q.dtype == k.dtype == v.dtype:
            lite3r_quantize_fp8_qkv(q, k, v, self.shape, self.q8, self.k8, self.v8, stream)
        else:
            lite3r_quantize_fp8(q, self.shape, self.q8, stream)
            lite3r_quantize_fp8(k, self.shape, self.k8, stream)
            lite3r_quantize_fp8(v, self.shape, self.v8, stream)

    def make_plan(self, stream=None):
        lite3r_sla_plan(self.q8, self.k8, self.shape, self.crit, self.neg, self.plan, stream)

    def forward(self, proj, stream=None, out=None):
        """out: optional result tensor of the engine's output shape (default: the engine's own ``out``)."""
        out = self.out if out is None else out
        lite3r_sla_forward(self.q8, self.k8, self.v8, proj, self.shape, self.phi,
                           None if self.plan_inside else self.plan, out, self.workspace, self.status, stream,
                           crit=self.crit, neg=self.neg)
        return out

    def run(self, q, k, v, proj, stream=None, out=None, overlap=False):
        """Quantise, plan, forward.  overlap=True runs the plan-independent first half of the forward (summaries, fp16
        V) on a side stream beside the plan kernel; the results are the same."""
        if self.plan_inside:
            self.quantize(q, k, v, stream)
            return self.forward(proj, stream, out)
        if not overlap or self.plan.k_marg == 0:
            self.quantize(q, k, v, stream)
            self.make_plan(stream)
            return self.forward(proj, stream, out)
        main = torch.cuda.current_stream(self.device) if stream is None else stream
        if self._side is None:
            self._side = torch.cuda.Stream(self.device)
        out = self.out if out is None else out
        self.quantize(q, k, v, main)
        self._side.wait_stream(main)  # codes and scales are ready
        lite3r_sla_forward_begin(self.k8, self.v8, proj, self.shape, self.phi, self.plan, self.workspace, self.status,
                                 self._side)
        self.make_plan(main)
        main.wait_stream(self._side)
        lite3r_sla_forward_finish(self.q8, self.k8, self.v8, self.shape, self.phi, self.plan, out, self.workspace,
                                  self.status, main)
        return out

    def run_graph(self, q, k, v, proj, out=None):
        """The same step (quantise, plan, forward with the overlapped first half) replayed as one CUDA graph on the
        current stream: the five kernel launches, the status clear and the stream fork / join of a step then cost one
        launch on the host, which is a tenth of the step at short sequences.  The graph is captured on first use for
        these tensors (and again when a tensor's address changes); results are identical to ``run``.  The library
        calls only enqueue work on the stream they are given and allocate nothing, which is what makes them
        capturable; call ``run`` once before (shared-memory limits and tensor maps are set up on first use)."""
        out = self.out if out is None else out
        key = (q.data_ptr(), k.data_ptr(), v.data_ptr(), proj.data_ptr(), out.data_ptr())
        if self._graph is None or self._graph[1] != key:
            self.run(q, k, v, proj, out=out, overlap=True)  # first-use set-up happens outside the capture
            torch.cuda.synchronize(self.device)
            graph = torch.cuda.CUDAGraph()
            capture_stream = torch.cuda.Stream(self.device)
            capture_stream.wait_stream(torch.cuda.current_stream(self.device))
            with torch.cuda.graph(graph, stream=capture_stream):
                self.run(q, k, v, proj, out=out, overlap=True)
            torch.cuda.current_stream(self.device).wait_stream(capture_stream)
            self._graph = (graph, key)
        self._graph[0].replay()
        return out

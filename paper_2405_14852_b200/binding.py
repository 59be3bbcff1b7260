"""ctypes binding of libpvt.so: argument marshalling only.

Every step of the V step (norms, selection, target formation, search, code
write, dequantisation) runs in the CUDA kernels behind the C ABI declared in
``include/pvt.h``; this module only turns torch tensors into pointers and sizes.
There is no CPU fallback: if the library cannot be loaded, or a call is rejected,
an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

from . import build as _build

PVT_F32, PVT_F16 = 0, 1
PVT_U8, PVT_U16 = 0, 1
PVT_OK, PVT_EINVAL, PVT_EUNSUPPORTED, PVT_EWORKSPACE, PVT_ECUDA, PVT_ETOOLARGE = 0, -1, -2, -3, -4, -5
PVT_NOALLOC_MAX_GROUPS = 1 << 21
PVT_DEV_BAD_INDEX, PVT_DEV_BAD_CODE, PVT_DEV_WAIT_EXPIRED, PVT_DEV_INTERNAL = 1, 2, 4, 8
PVT_KERNEL_SELECT, PVT_KERNEL_ENCODE_MAIN, PVT_KERNEL_ENCODE_AUX, PVT_KERNEL_DEQUANT = 0, 1, 2, 3
PVT_KERNEL_ENCODE_RESCORE = 4
PVT_KERNEL_PSTEP_GRAD, PVT_KERNEL_ADAM, PVT_KERNEL_TRUST, PVT_KERNEL_REFINE = 5, 6, 7, 8
PVT_M1_AUTO, PVT_M1_FP32, PVT_M1_TENSOR = 0, 1, 2
PVT_SAMPLE_UNIFORM, PVT_SAMPLE_PROPORTIONAL = 0, 1


class pvt_layer(ctypes.Structure):
    _fields_ = [
        ("rows", ctypes.c_int32), ("cols", ctypes.c_int32), ("group_dim", ctypes.c_int32),
        ("num_codebooks", ctypes.c_int32), ("codebook_size", ctypes.c_int32),
        ("codebook_dtype", ctypes.c_int32), ("code_dtype", ctypes.c_int32), ("beam", ctypes.c_int32),
        ("eta", ctypes.c_float), ("reserved_", ctypes.c_int32),
        ("W", ctypes.c_void_p), ("g", ctypes.c_void_p), ("scale", ctypes.c_void_p),
        ("codebooks", ctypes.c_void_p), ("codes", ctypes.c_void_p),
    ]


class PvtError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: {strerror(code)} (code {code})" + (f": {last_cuda_error()}" if code == PVT_ECUDA else ""))
        self.code = code


_lib = None


def library_path() -> str:
    return _build.LIB


def lib():
    """The loaded C library.  Builds it in-tree if nvcc is available and the
    shared object is missing or stale; raises if it cannot be loaded."""
    global _lib
    if _lib is None:
        path = library_path()
        if _build.needs_build():
            try:
                _build.build()
            except Exception as exc:  # no compiler on this machine: use the shipped object if there is one
                if not os.path.exists(path):
                    raise RuntimeError(f"libpvt.so is missing and could not be built: {exc}") from exc
        L = ctypes.CDLL(path)
        vp, u64, sz, fl = ctypes.c_void_p, ctypes.c_uint64, ctypes.c_size_t, ctypes.c_float
        lp = ctypes.POINTER(pvt_layer)
        L.pvt_workspace_bytes.restype = sz
        L.pvt_workspace_bytes.argtypes = [lp, u64]
        L.pvt_workspace_init.restype = ctypes.c_int
        L.pvt_workspace_init.argtypes = [vp, sz, vp]
        L.pvt_vstep_select.restype = ctypes.c_int
        L.pvt_vstep_select.argtypes = [lp, u64, vp, vp, sz, vp]
        L.pvt_vstep_select_noalloc.restype = ctypes.c_int
        L.pvt_vstep_select_noalloc.argtypes = [lp, u64, vp, vp, vp]
        L.pvt_vstep_select_ste.restype = ctypes.c_int
        L.pvt_vstep_select_ste.argtypes = [lp, vp, u64, vp, vp, sz, vp]
        L.pvt_vstep_sample.restype = ctypes.c_int
        L.pvt_vstep_sample.argtypes = [lp, u64, ctypes.c_int32, u64, vp, vp, sz, vp]
        L.pvt_vstep_encode.restype = ctypes.c_int
        L.pvt_vstep_encode.argtypes = [lp, vp, u64, vp, vp, sz, vp]
        L.pvt_trust_workspace_bytes.restype = sz
        L.pvt_trust_workspace_bytes.argtypes = [lp, u64]
        L.pvt_vstep_trust.restype = ctypes.c_int
        L.pvt_vstep_trust.argtypes = [lp, u64, fl, vp, vp, vp, vp, sz, vp]
        L.pvt_vstep_refine.restype = ctypes.c_int
        L.pvt_vstep_refine.argtypes = [lp, vp, u64, ctypes.c_int32, vp, vp, vp, vp]
        L.pvt_block_workspace_bytes.restype = sz
        L.pvt_block_workspace_bytes.argtypes = [lp, ctypes.POINTER(u64), ctypes.c_int32]
        L.pvt_vstep_block.restype = ctypes.c_int
        L.pvt_vstep_block.argtypes = [lp, ctypes.POINTER(u64), ctypes.c_int32, ctypes.POINTER(vp), ctypes.POINTER(vp),
                                      ctypes.c_int32, vp, sz, vp]
        L.pvt_dequant.restype = ctypes.c_int
        L.pvt_dequant.argtypes = [lp, vp, ctypes.c_int32, vp, vp]
        L.pvt_pstep_grad.restype = ctypes.c_int
        L.pvt_pstep_grad.argtypes = [lp, vp, vp, vp, vp]
        L.pvt_adam_update.restype = ctypes.c_int
        L.pvt_adam_update.argtypes = [vp, vp, vp, vp, vp, u64, fl, fl, fl, fl, fl, fl, vp]
        L.pvt_adam_direction.restype = ctypes.c_int
        L.pvt_adam_direction.argtypes = [vp, vp, vp, vp, u64, fl, fl, fl, fl, fl, vp]
        L.pvt_adam_bias.restype = ctypes.c_int
        L.pvt_adam_bias.argtypes = [u64, fl, fl, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_float)]
        L.pvt_test_wait_limit.restype = None
        L.pvt_test_wait_limit.argtypes = [ctypes.c_uint32, ctypes.c_int64]
        L.pvt_status.restype = ctypes.c_int
        L.pvt_status.argtypes = [vp, vp]
        L.pvt_strerror.restype = ctypes.c_char_p
        L.pvt_strerror.argtypes = [ctypes.c_int]
        L.pvt_last_cuda_error.restype = ctypes.c_char_p
        L.pvt_version.restype = ctypes.c_int
        L.pvt_set_m1_search.restype = None
        L.pvt_set_m1_search.argtypes = [ctypes.c_int]
        L.pvt_timing_enable.restype = None
        L.pvt_timing_enable.argtypes = [ctypes.c_int]
        L.pvt_probe_fp32_tflops.restype = ctypes.c_int
        L.pvt_probe_fp32_tflops.argtypes = [vp, sz, ctypes.POINTER(ctypes.c_float), vp]
        L.pvt_launch_count.restype = ctypes.c_ulonglong
        L.pvt_timing_read.restype = ctypes.c_int
        L.pvt_timing_read.argtypes = [ctypes.c_int, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_int)]
        _lib = L
    return _lib


def strerror(code: int) -> str:
    return lib().pvt_strerror(code).decode()


def last_cuda_error() -> str:
    return lib().pvt_last_cuda_error().decode()


def _check(code: int, what: str) -> None:
    if code != PVT_OK:
        raise PvtError(code, what)


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def make_layer(rows: int, cols: int, W, g, scale, codebooks, codes, *, eta: float = 1.0, beam: int = 8,
               group_dim: int = 8) -> pvt_layer:
    """Describe a layer whose arrays are CUDA tensors (any of W, g, scale may be
    None for calls that do not read them).  codebooks: [M, K, 8] float32/float16;
    codes: [G, M] uint8/uint16."""
    M, K = int(codebooks.shape[0]), int(codebooks.shape[1])
    for t in (W, g, scale, codebooks, codes):
        if t is not None and (not t.is_cuda or not t.is_contiguous()):
            raise ValueError("layer tensors must be contiguous CUDA tensors")
    cb_dtype = {torch.float32: PVT_F32, torch.float16: PVT_F16}[codebooks.dtype]
    code_dtype = {torch.uint8: PVT_U8, torch.uint16: PVT_U16, torch.int16: PVT_U16}[codes.dtype]
    return pvt_layer(rows, cols, group_dim, M, K, cb_dtype, code_dtype, beam, float(eta), 0,
                     _ptr(W), _ptr(g), _ptr(scale), _ptr(codebooks), _ptr(codes))


def pvt_workspace_bytes(layer: pvt_layer, k: int) -> int:
    n = int(lib().pvt_workspace_bytes(ctypes.byref(layer), k))
    if n == 0:
        raise PvtError(PVT_EINVAL, "pvt_workspace_bytes")
    return n


def pvt_workspace_init(ws: torch.Tensor, stream=None) -> None:
    _check(lib().pvt_workspace_init(ws.data_ptr(), ws.numel() * ws.element_size(), _stream_ptr(stream)),
           "pvt_workspace_init")


def new_workspace(layer: pvt_layer, k: int, device=None) -> torch.Tensor:
    ws = torch.empty(pvt_workspace_bytes(layer, k), dtype=torch.uint8, device=device or "cuda")
    pvt_workspace_init(ws)
    return ws


def pvt_vstep_select(layer: pvt_layer, k: int, idx_out: torch.Tensor, ws: torch.Tensor, stream=None) -> None:
    _check(lib().pvt_vstep_select(ctypes.byref(layer), k, idx_out.data_ptr(), ws.data_ptr(),
                                  ws.numel() * ws.element_size(), _stream_ptr(stream)), "pvt_vstep_select")


def pvt_vstep_select_noalloc(layer: pvt_layer, k: int, idx_out: torch.Tensor,
                             status_out: Optional[torch.Tensor] = None, stream=None) -> None:
    """pvt_vstep_select without a workspace argument: for callers that cannot
    allocate device memory (frozen memory pool, host application owning the
    device memory, allocator-free thread).  The scratch is a fixed array inside
    the library, so the layer may have at most PVT_NOALLOC_MAX_GROUPS groups, and
    calls that could overlap on the GPU must be ordered by the caller."""
    _check(lib().pvt_vstep_select_noalloc(ctypes.byref(layer), k, idx_out.data_ptr(), _ptr(status_out),
                                          _stream_ptr(stream)), "pvt_vstep_select_noalloc")


def pvt_vstep_select_ste(layer: pvt_layer, buffer: torch.Tensor, k: int, idx_out: torch.Tensor, ws: torch.Tensor,
                         stream=None) -> None:
    """pvt_vstep_select that also lets the straight-through buffer (float32 [rows, cols], in place) take the
    step -eta * g (Appendix E)."""
    if buffer.dtype != torch.float32 or not buffer.is_cuda or not buffer.is_contiguous():
        raise ValueError("buffer must be a contiguous float32 CUDA tensor")
    _check(lib().pvt_vstep_select_ste(ctypes.byref(layer), buffer.data_ptr(), k, idx_out.data_ptr(), ws.data_ptr(),
                                      ws.numel() * ws.element_size(), _stream_ptr(stream)), "pvt_vstep_select_ste")


def pvt_vstep_sample(layer: pvt_layer, k: int, rule: int, seed: int, idx_out: torch.Tensor, ws: torch.Tensor,
                     stream=None) -> None:
    """A random subspace of k groups: PVT_SAMPLE_UNIFORM or PVT_SAMPLE_PROPORTIONAL (to the squared update norm)."""
    _check(lib().pvt_vstep_sample(ctypes.byref(layer), k, rule, seed, idx_out.data_ptr(), ws.data_ptr(),
                                  ws.numel() * ws.element_size(), _stream_ptr(stream)), "pvt_vstep_sample")


def pvt_vstep_encode(layer: pvt_layer, idx: torch.Tensor, k: int, err_out: Optional[torch.Tensor],
                     ws: torch.Tensor, stream=None) -> None:
    _check(lib().pvt_vstep_encode(ctypes.byref(layer), idx.data_ptr(), k, _ptr(err_out), ws.data_ptr(),
                                  ws.numel() * ws.element_size(), _stream_ptr(stream)), "pvt_vstep_encode")


def pvt_trust_workspace_bytes(layer: pvt_layer, k_max: int) -> int:
    n = int(lib().pvt_trust_workspace_bytes(ctypes.byref(layer), k_max))
    if n == 0:
        raise PvtError(PVT_EINVAL, "pvt_trust_workspace_bytes")
    return n


def new_trust_workspace(layer: pvt_layer, k_max: int, device=None) -> torch.Tensor:
    ws = torch.empty(pvt_trust_workspace_bytes(layer, k_max), dtype=torch.uint8, device=device or "cuda")
    pvt_workspace_init(ws)
    return ws


def pvt_vstep_trust(layer: pvt_layer, k_max: int, ratio: float, idx_out: torch.Tensor, n_out: torch.Tensor,
                    stats_out: Optional[torch.Tensor], ws: torch.Tensor, stream=None) -> None:
    """V step with the subspace size taken from the trust ratio: idx_out (uint32 [k_max]) receives the groups in
    rank order, n_out (one int64/uint64) how many of them keep their new codes, stats_out (float64 [2] or None)
    the squared norm of the dequantised matrix before and the squared change that was kept."""
    _check(lib().pvt_vstep_trust(ctypes.byref(layer), k_max, ratio, idx_out.data_ptr(), n_out.data_ptr(),
                                 _ptr(stats_out), ws.data_ptr(), ws.numel() * ws.element_size(),
                                 _stream_ptr(stream)), "pvt_vstep_trust")


def pvt_vstep_refine(layer: pvt_layer, idx: torch.Tensor, k: int, max_moves: int,
                     err_out: Optional[torch.Tensor] = None, moves_out: Optional[torch.Tensor] = None,
                     status: Optional[torch.Tensor] = None, stream=None) -> None:
    """Local search over single-code changes (Appendix D) on the listed groups, from the stored codes."""
    _check(lib().pvt_vstep_refine(ctypes.byref(layer), idx.data_ptr(), k, max_moves, _ptr(err_out), _ptr(moves_out),
                                  _ptr(status), _stream_ptr(stream)), "pvt_vstep_refine")


def pvt_dequant(layer: pvt_layer, W_hat: torch.Tensor, status: Optional[torch.Tensor] = None, stream=None) -> None:
    out_dtype = {torch.float32: PVT_F32, torch.float16: PVT_F16}[W_hat.dtype]
    _check(lib().pvt_dequant(ctypes.byref(layer), W_hat.data_ptr(), out_dtype, _ptr(status), _stream_ptr(stream)),
           "pvt_dequant")


class Block:
    """Host arrays for pvt_vstep_block: the layers of one model block, their subspace sizes and output pointers
    (marshalled once; the tensors must stay alive while the block is used)."""

    def __init__(self, layers, ks, idx_outs, W_hats=None):
        n = len(layers)
        self.n = n
        self.layers = (pvt_layer * n)(*layers)
        self.k = (ctypes.c_uint64 * n)(*[int(x) for x in ks])
        self.idx = (ctypes.c_void_p * n)(*[t.data_ptr() for t in idx_outs])
        self.W_hat = None
        self.out_dtype = PVT_F32
        if W_hats is not None:
            self.W_hat = (ctypes.c_void_p * n)(*[None if t is None else t.data_ptr() for t in W_hats])
            dts = {t.dtype for t in W_hats if t is not None}
            if len(dts) > 1:
                raise ValueError("the dequantised matrices of a block share one dtype")
            if dts:
                self.out_dtype = {torch.float32: PVT_F32, torch.float16: PVT_F16}[dts.pop()]
        self._keep = (list(idx_outs), list(W_hats) if W_hats is not None else None)

    def workspace_bytes(self) -> int:
        need = int(lib().pvt_block_workspace_bytes(self.layers, self.k, self.n))
        if need == 0:
            raise PvtError(PVT_EINVAL, "pvt_block_workspace_bytes")
        return need


def pvt_vstep_block(block: Block, ws: torch.Tensor, stream=None) -> None:
    """select -> encode -> dequantise over every layer of the block, one C call."""
    _check(lib().pvt_vstep_block(block.layers, block.k, block.n, block.idx, block.W_hat, block.out_dtype, ws.data_ptr(),
                                 ws.numel() * ws.element_size(), _stream_ptr(stream)), "pvt_vstep_block")


def pvt_pstep_grad(layer: pvt_layer, grad_codebooks: torch.Tensor, grad_scale: Optional[torch.Tensor] = None,
                   status: Optional[torch.Tensor] = None, stream=None) -> None:
    """grad_codebooks [M, K, 8] float64, grad_scale [rows] float64 or None (both overwritten)."""
    assert grad_codebooks.dtype == torch.float64 and (grad_scale is None or grad_scale.dtype == torch.float64)
    _check(lib().pvt_pstep_grad(ctypes.byref(layer), grad_codebooks.data_ptr(), _ptr(grad_scale), _ptr(status),
                                _stream_ptr(stream)), "pvt_pstep_grad")


def pvt_adam_bias(step: int, beta1: float, beta2: float):
    """Bias corrections 1 - beta^t of step t >= 1 as the binary32 numbers pvt_adam_update takes."""
    b1, b2 = ctypes.c_float(0.0), ctypes.c_float(0.0)
    _check(lib().pvt_adam_bias(step, beta1, beta2, ctypes.byref(b1), ctypes.byref(b2)), "pvt_adam_bias")
    return b1.value, b2.value


def pvt_adam_update(param: torch.Tensor, grad: torch.Tensor, exp_avg: torch.Tensor, exp_avg_sq: torch.Tensor,
                    step: int, lr: float, beta1: float = 0.9, beta2: float = 0.95, eps: float = 1e-8,
                    param_f16: Optional[torch.Tensor] = None, stream=None) -> None:
    """One Adam update in place (param, exp_avg, exp_avg_sq float32; grad float64; optional float16 copy)."""
    assert param.dtype == torch.float32 and grad.dtype == torch.float64
    assert exp_avg.dtype == torch.float32 and exp_avg_sq.dtype == torch.float32
    assert param_f16 is None or param_f16.dtype == torch.float16
    bias1, bias2 = pvt_adam_bias(step, beta1, beta2)
    _check(lib().pvt_adam_update(param.data_ptr(), _ptr(param_f16), grad.data_ptr(), exp_avg.data_ptr(),
                                 exp_avg_sq.data_ptr(), param.numel(), lr, beta1, beta2, eps, bias1, bias2,
                                 _stream_ptr(stream)), "pvt_adam_update")


def pvt_adam_direction(grad: torch.Tensor, exp_avg: torch.Tensor, exp_avg_sq: torch.Tensor, out: torch.Tensor,
                       step: int, beta1: float = 0.9, beta2: float = 0.95, eps: float = 1e-8, stream=None) -> None:
    """Adam-normalised update direction of the V step (all float32; moments updated in place)."""
    for t in (grad, exp_avg, exp_avg_sq, out):
        assert t.dtype == torch.float32 and t.is_contiguous()
    bias1, bias2 = pvt_adam_bias(step, beta1, beta2)
    _check(lib().pvt_adam_direction(grad.data_ptr(), exp_avg.data_ptr(), exp_avg_sq.data_ptr(), out.data_ptr(),
                                    grad.numel(), beta1, beta2, eps, bias1, bias2, _stream_ptr(stream)),
           "pvt_adam_direction")


def pvt_status(ws: torch.Tensor, stream=None) -> int:
    rc = int(lib().pvt_status(ws.data_ptr(), _stream_ptr(stream)))
    if rc < 0:
        raise PvtError(rc, "pvt_status")
    return rc


def pvt_version() -> int:
    return int(lib().pvt_version())


def pvt_set_m1_search(mode: int) -> None:
    """Engine of the single-codebook search: PVT_M1_AUTO, PVT_M1_FP32 or PVT_M1_TENSOR."""
    lib().pvt_set_m1_search(mode)


def pvt_probe_fp32_tflops(stream=None) -> float:
    """Measured FP32 FMA throughput of the current device in TFLOP/s (a short kernel of independent FMA chains)."""
    props = torch.cuda.get_device_properties(torch.cuda.current_device())
    scratch = torch.empty(props.multi_processor_count * 2048, dtype=torch.float32, device="cuda")
    out = ctypes.c_float(0.0)
    _check(lib().pvt_probe_fp32_tflops(scratch.data_ptr(), scratch.numel(), ctypes.byref(out), _stream_ptr(stream)),
           "pvt_probe_fp32_tflops")
    return float(out.value)


def pvt_test_wait_limit(max_polls: int = 0, withhold_copy: int = -1) -> None:
    """Test hook: poll limit of the search kernels' on-chip waits (0 = default) and the sequence number of a
    codebook copy that every thread block leaves out (-1 = none).  Process-wide."""
    lib().pvt_test_wait_limit(max_polls, withhold_copy)


def pvt_launch_count() -> int:
    return int(lib().pvt_launch_count())


def pvt_timing_enable(on: bool) -> None:
    lib().pvt_timing_enable(1 if on else 0)


def pvt_timing_read(kernel_id: int):
    """(total milliseconds, launches) of one kernel class since the last read."""
    ms, n = ctypes.c_float(0.0), ctypes.c_int(0)
    _check(lib().pvt_timing_read(kernel_id, ctypes.byref(ms), ctypes.byref(n)), "pvt_timing_read")
    return float(ms.value), int(n.value)

"""ctypes binding of the C ABI (include/cubicquant.h).  Argument marshalling only."""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.environ.get("CUBICQUANT_LIB") or os.path.join(_HERE, "libcubicquant.so")

CQ_MODEL_DTYPE = 0
CQ_DYN_A8 = 1

_lib = None


class CubicQuantError(RuntimeError):
    pass


def library_path() -> str:
    return _LIB_PATH


def lib():
    """The loaded shared library.  Fails loudly when it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise CubicQuantError(f"{_LIB_PATH} is missing: build it with `python -m paper_2608_06763_b200.build` "
                                  "(there is no fallback path)")
        L = C.CDLL(_LIB_PATH)
        vp, i, i64, sz = C.c_void_p, C.c_int, C.c_int64, C.c_size_t
        L.cq_status_string.restype = C.c_char_p
        L.cq_status_string.argtypes = [i]
        L.cq_last_cuda_error.restype = i
        L.cq_canonical_code_bytes.restype = sz
        L.cq_canonical_code_bytes.argtypes = [i, i64, i64]
        L.cq_effective_bits.restype = C.c_double
        L.cq_effective_bits.argtypes = [i, i]
        L.cq_layout_bytes.restype = sz
        L.cq_layout_bytes.argtypes = [i, i, i64, i64]
        L.cq_workspace_bytes.restype = sz
        L.cq_workspace_bytes.argtypes = [i, i, i64, i64, i64, i]
        L.cq_workspace_init.argtypes = [vp, sz, vp]
        L.cq_pack_codes.argtypes = [vp, i, i64, i64, vp, vp]
        L.cq_repack.argtypes = [vp, vp, vp, vp, i, i, i64, i64, vp, vp]
        L.cq_unpack.argtypes = [vp, i, i, i64, i64, vp, vp, vp, vp, vp]
        L.cq_gemm.argtypes = [vp, i, i, vp, vp, i64, i64, i64, i, vp, sz, vp]
        L.cq_gemm_f16.argtypes = [vp, i, i, vp, vp, i64, i64, i64, i, vp, sz, vp]
        L.cq_quantize_a8_f16.argtypes = [vp, i64, i64, vp, vp, vp]
        L.cq_mlp_workspace_bytes.restype = sz
        L.cq_mlp_workspace_bytes.argtypes = [i, i, i, i, i64, i64, i64, i64, i]
        L.cq_mlp_swiglu.argtypes = [vp, i, i, vp, i, i, vp, vp, i64, i64, i64, i64, i, i, vp, sz, vp]
        L.cq_mlp_swiglu.restype = i
        L.cq_routed_workspace_bytes.restype = sz
        L.cq_routed_workspace_bytes.argtypes = [i, i, i, vp, i64, i64, i]
        L.cq_gemm_routed.argtypes = [vp, i, i, i, vp, vp, vp, vp, i64, i64, i64, i, i, vp, sz, vp]
        L.cq_gemm_routed.restype = i
        L.cq_gemm_status.argtypes = [vp, sz, vp]
        L.cq_gemm_status.restype = i
        L.cq_gemv_static.argtypes = [vp, i, i, vp, vp, i64, i64, i64, vp]
        L.cq_gemv_static.restype = i
        L.cq_gemm_host.argtypes = [vp, i, i, vp, vp, vp, vp, i64, i64, i64, i, vp, sz, vp]
        L.cq_quantize_a8.argtypes = [vp, i64, i64, vp, vp, vp]
        L.cq_decode_levels.argtypes = [vp, i, i, i64, i64, vp, vp]
        L.cq_decode_carriers.argtypes = [vp, i, i, i64, i64, vp, vp]
        L.cq_decode_weights.argtypes = [vp, i, i, i64, i64, vp, vp]
        L.cq_debug_a8_partials.argtypes = [vp, i, i, vp, i64, i64, i64, vp, vp]
        L.cq_debug_gemm_plan.argtypes = [i, i, i64, i64, i64, i, vp]
        L.cq_debug_gemm_plan.restype = i
        L.cq_debug_wait_timeout.argtypes = [vp, sz, i64, vp]
        L.cq_debug_wait_timeout.restype = i
        L.cq_encode_assign.argtypes = [vp, i, i, i64, i64, vp, vp, vp, i, vp, vp]
        L.cq_encode_scale.argtypes = [vp, vp, i, i, i64, i64, vp, vp, i, vp, vp]
        L.cq_encode_losses.argtypes = [vp, vp, i, i, i64, i64, vp, vp, vp, vp, vp, vp]
        L.cq_encode.argtypes = [vp, i, i, i64, i64, i, i, vp, vp, vp, vp, vp]
        for name in ("cq_workspace_init", "cq_pack_codes", "cq_repack", "cq_unpack", "cq_gemm", "cq_gemm_f16", "cq_gemm_host",
                     "cq_quantize_a8", "cq_quantize_a8_f16", "cq_decode_levels", "cq_decode_carriers", "cq_decode_weights",
                     "cq_debug_a8_partials", "cq_encode_assign", "cq_encode_scale", "cq_encode_losses", "cq_encode"):
            getattr(L, name).restype = i
        _lib = L
    return _lib


def _check(status: int, what: str):
    if status != 0:
        L = lib()
        raise CubicQuantError(f"{what}: {L.cq_status_string(status).decode()} (cuda error {L.cq_last_cuda_error()})")


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t: torch.Tensor) -> int:
    assert t.is_cuda and t.is_contiguous(), "device, contiguous tensors only"
    return t.data_ptr()


def cq_status_string(status: int) -> str:
    return lib().cq_status_string(status).decode()


def cq_canonical_code_bytes(B, N, K) -> int:
    return lib().cq_canonical_code_bytes(B, N, K)


def cq_effective_bits(B, G) -> float:
    return lib().cq_effective_bits(B, G)


def cq_layout_bytes(B, G, N, K) -> int:
    return lib().cq_layout_bytes(B, G, N, K)


def cq_workspace_bytes(B, G, M, N, K, mode) -> int:
    return lib().cq_workspace_bytes(B, G, M, N, K, mode)


def cq_workspace_init(workspace: torch.Tensor):
    _check(lib().cq_workspace_init(_ptr(workspace), workspace.numel() * workspace.element_size(), _stream()),
           "cq_workspace_init")


def cq_pack_codes(k: torch.Tensor, B: int) -> torch.Tensor:
    """int8 logical codes [N, K] -> canonical packed bytes [N, ceil(K*B/8)] (uint8, device)."""
    N, K = k.shape
    out = torch.empty((N, (K * B + 7) // 8), dtype=torch.uint8, device=k.device)
    _check(lib().cq_pack_codes(_ptr(k), B, N, K, _ptr(out), _stream()), "cq_pack_codes")
    return out


@dataclass
class PackedWeights:
    """A matrix in the device layout (owned torch buffer plus its format)."""
    layout: torch.Tensor
    B: int
    G: int
    N: int
    K: int


def cq_repack(codes, scale, a, b, B, G, N, K) -> PackedWeights:
    """Canonical tensors (device: codes uint8, scale fp32, a/b fp16) -> device layout."""
    nbytes = cq_layout_bytes(B, G, N, K)
    if nbytes == 0:
        _check(lib().cq_repack(0, 0, 0, 0, B, G, N, K, 0, 0) or -2, "cq_repack")
    layout = torch.empty(nbytes, dtype=torch.uint8, device=codes.device)
    _check(lib().cq_repack(_ptr(codes), _ptr(scale), _ptr(a), _ptr(b), B, G, N, K, _ptr(layout), _stream()),
           "cq_repack")
    return PackedWeights(layout, B, G, N, K)


def cq_unpack(pw: PackedWeights):
    dev = pw.layout.device
    codes = torch.empty((pw.N, (pw.K * pw.B + 7) // 8), dtype=torch.uint8, device=dev)
    ng = pw.K // pw.G
    scale = torch.empty((pw.N, ng), dtype=torch.float32, device=dev)
    a = torch.empty((pw.N, ng), dtype=torch.float16, device=dev)
    b = torch.empty((pw.N, ng), dtype=torch.float16, device=dev)
    _check(lib().cq_unpack(_ptr(pw.layout), pw.B, pw.G, pw.N, pw.K, _ptr(codes), _ptr(scale), _ptr(a), _ptr(b),
                           _stream()), "cq_unpack")
    return codes, scale, a, b


def cq_gemm(pw: PackedWeights, x: torch.Tensor, mode: int = CQ_MODEL_DTYPE, workspace: torch.Tensor | None = None,
            out: torch.Tensor | None = None) -> torch.Tensor:
    """y[M, N] = x[M, K] * What^T from the packed weights; x is bf16 or fp16 (the model dtype), y has the same dtype."""
    assert x.dtype in (torch.bfloat16, torch.float16) and x.dim() == 2 and x.shape[1] == pw.K
    M = x.shape[0]
    if workspace is None:
        workspace = torch.zeros(cq_workspace_bytes(pw.B, pw.G, M, pw.N, pw.K, mode), dtype=torch.uint8, device=x.device)
    y = out if out is not None else torch.empty((M, pw.N), dtype=x.dtype, device=x.device)
    assert y.dtype == x.dtype
    fn = lib().cq_gemm if x.dtype == torch.bfloat16 else lib().cq_gemm_f16
    _check(fn(_ptr(pw.layout), pw.B, pw.G, _ptr(x), _ptr(y), M, pw.N, pw.K, mode, _ptr(workspace),
                         workspace.numel(), _stream()), "cq_gemm")
    return y


def cq_mlp_swiglu(gate_up: PackedWeights, down: PackedWeights, x: torch.Tensor, mode_gate_up: int = CQ_MODEL_DTYPE,
                  workspace: torch.Tensor | None = None, out: torch.Tensor | None = None) -> torch.Tensor:
    """y[M, N] = down(silu(gate) * up) with (gate | up) = gate_up(x): the SwiGLU MLP block whose activation and
    Dynamic-A8 quantiser in front of the down projection are one kernel.  gate_up is 2 I x K, down is N x I."""
    assert x.dtype in (torch.bfloat16, torch.float16) and x.dim() == 2 and x.shape[1] == gate_up.K
    M, K, I, N = x.shape[0], gate_up.K, down.K, down.N
    assert gate_up.N == 2 * I
    need = lib().cq_mlp_workspace_bytes(gate_up.B, gate_up.G, down.B, down.G, M, K, I, N, mode_gate_up)
    if workspace is None:
        workspace = torch.zeros(need, dtype=torch.uint8, device=x.device)
    y = out if out is not None else torch.empty((M, N), dtype=x.dtype, device=x.device)
    _check(lib().cq_mlp_swiglu(_ptr(gate_up.layout), gate_up.B, gate_up.G, _ptr(down.layout), down.B, down.G, _ptr(x), _ptr(y),
                               M, K, I, N, mode_gate_up, 1 if x.dtype == torch.float16 else 0, _ptr(workspace),
                               workspace.numel(), _stream()), "cq_mlp_swiglu")
    return y


def cq_gemm_routed(experts, x: torch.Tensor, route_token: torch.Tensor, expert_offset, mode: int = CQ_MODEL_DTYPE,
                   workspace: torch.Tensor | None = None) -> torch.Tensor:
    """Route-major y[R, N]: route r multiplies token route_token[r] of x by the matrix whose block
    [expert_offset[e], expert_offset[e+1]) holds r.  experts: list of PackedWeights of one shape and format;
    route_token: int32 device tensor [R]; expert_offset: E + 1 host integers."""
    E = len(experts)
    p0 = experts[0]
    assert all((p.B, p.G, p.N, p.K) == (p0.B, p0.G, p0.N, p0.K) for p in experts)
    assert x.dtype in (torch.bfloat16, torch.float16) and x.dim() == 2 and x.shape[1] == p0.K
    assert route_token.dtype == torch.int32 and route_token.is_cuda
    off = (C.c_int64 * (E + 1))(*[int(v) for v in expert_offset])
    ptrs = (C.c_void_p * E)(*[_ptr(p.layout) for p in experts])
    R = int(expert_offset[-1])
    assert route_token.numel() == R
    need = lib().cq_routed_workspace_bytes(p0.B, p0.G, E, off, p0.N, p0.K, mode)
    if workspace is None:
        workspace = torch.zeros(max(need, 512), dtype=torch.uint8, device=x.device)
    y = torch.empty((R, p0.N), dtype=x.dtype, device=x.device)
    _check(lib().cq_gemm_routed(ptrs, E, p0.B, p0.G, _ptr(x), _ptr(route_token), off, _ptr(y), x.shape[0], p0.N, p0.K, mode,
                                1 if x.dtype == torch.float16 else 0, _ptr(workspace), workspace.numel(), _stream()),
           "cq_gemm_routed")
    return y


def cq_gemm_status(workspace: torch.Tensor) -> int:
    """0, or the negative CQ_ERR_TIMEOUT when a bounded device wait gave up (synchronises the stream)."""
    return lib().cq_gemm_status(_ptr(workspace), workspace.numel(), _stream())


def cq_gemv_static(pw: PackedWeights, x: torch.Tensor, out: torch.Tensor | None = None) -> torch.Tensor:
    """Small-M product (M <= 16, model dtype) that takes its scratch from the array built into the
    library: for callers that may not allocate.  Calls on one device must not overlap."""
    assert x.dtype == torch.bfloat16 and x.dim() == 2 and x.shape[1] == pw.K
    M = x.shape[0]
    y = out if out is not None else torch.empty((M, pw.N), dtype=torch.bfloat16, device=x.device)
    _check(lib().cq_gemv_static(_ptr(pw.layout), pw.B, pw.G, _ptr(x), _ptr(y), M, pw.N, pw.K, _stream()),
           "cq_gemv_static")
    return y


def cq_gemm_host(pw: PackedWeights, x_host: torch.Tensor, y_host: torch.Tensor, x_dev: torch.Tensor,
                 y_dev: torch.Tensor, mode: int, workspace: torch.Tensor):
    """Host-buffer variant: copies x in, runs the product, copies y out, waits."""
    M = x_host.shape[0]
    assert not x_host.is_cuda and not y_host.is_cuda
    _check(lib().cq_gemm_host(_ptr(pw.layout), pw.B, pw.G, x_host.data_ptr(), y_host.data_ptr(), _ptr(x_dev),
                              _ptr(y_dev), M, pw.N, pw.K, mode, _ptr(workspace), workspace.numel(), _stream()),
           "cq_gemm_host")
    return y_host


def cq_quantize_a8(x: torch.Tensor):
    M, K = x.shape
    x8 = torch.empty((M, K), dtype=torch.int8, device=x.device)
    dx = torch.empty(M, dtype=torch.float32, device=x.device)
    fn = lib().cq_quantize_a8 if x.dtype == torch.bfloat16 else lib().cq_quantize_a8_f16
    _check(fn(_ptr(x), M, K, _ptr(x8), _ptr(dx), _stream()), "cq_quantize_a8")
    return x8, dx


def _num_levels(B):
    return 1 if B == 1 else 1 << (B - 1)


def cq_decode_levels(pw: PackedWeights) -> torch.Tensor:
    out = torch.empty((pw.N, pw.K // pw.G, _num_levels(pw.B)), dtype=torch.float32, device=pw.layout.device)
    _check(lib().cq_decode_levels(_ptr(pw.layout), pw.B, pw.G, pw.N, pw.K, _ptr(out), _stream()), "cq_decode_levels")
    return out


def cq_decode_carriers(pw: PackedWeights) -> torch.Tensor:
    out = torch.empty((pw.N, pw.K // pw.G, _num_levels(pw.B)), dtype=torch.int8, device=pw.layout.device)
    _check(lib().cq_decode_carriers(_ptr(pw.layout), pw.B, pw.G, pw.N, pw.K, _ptr(out), _stream()),
           "cq_decode_carriers")
    return out


def cq_decode_weights(pw: PackedWeights) -> torch.Tensor:
    out = torch.empty((pw.N, pw.K), dtype=torch.float32, device=pw.layout.device)
    _check(lib().cq_decode_weights(_ptr(pw.layout), pw.B, pw.G, pw.N, pw.K, _ptr(out), _stream()),
           "cq_decode_weights")
    return out


def cq_debug_a8_partials(pw: PackedWeights, x8: torch.Tensor) -> torch.Tensor:
    M = x8.shape[0]
    out = torch.empty((M, pw.N, pw.K // pw.G), dtype=torch.int32, device=x8.device)
    _check(lib().cq_debug_a8_partials(_ptr(pw.layout), pw.B, pw.G, _ptr(x8), M, pw.N, pw.K, _ptr(out), _stream()),
           "cq_debug_a8_partials")
    return out


def cq_debug_gemm_plan(B: int, G: int, M: int, N: int, K: int, mode: int = CQ_MODEL_DTYPE) -> dict:
    """How the large-M GEMM of `mode` (M > 16) spreads a problem over the current device."""
    out = (C.c_int64 * 5)()
    _check(lib().cq_debug_gemm_plan(B, G, M, N, K, mode, out), "cq_debug_gemm_plan")
    return {"token_tile": out[0], "whole_tile_ctas": out[1], "stream_k_ctas": out[2], "stream_k_tiles": out[3],
            "runs_cross_tiles": bool(out[4])}


def cq_debug_wait_timeout(workspace: torch.Tensor, limit_cycles: int = 2_000_000):
    """One bounded wait that runs out (about a millisecond by default); the workspace's status word records it."""
    _check(lib().cq_debug_wait_timeout(_ptr(workspace), workspace.numel() * workspace.element_size(), limit_cycles,
                                       _stream()), "cq_debug_wait_timeout")


CQ_FIT_CONTINUOUS, CQ_FIT_JOINT = 0, 1
CQ_EFFORT = {"int_absmax": 0, "int_clipped": 1, "fast": 2, "reference": 3}


def cq_encode_assign(W: torch.Tensor, B: int, G: int, scale, a, b, objective: int = CQ_FIT_CONTINUOUS) -> torch.Tensor:
    """W float32 [N, K]; scale float32, a / b float16 [N, K/G] -> signed codes int8 [N, K]."""
    N, K = W.shape
    k = torch.empty((N, K), dtype=torch.int8, device=W.device)
    _check(lib().cq_encode_assign(_ptr(W), B, G, N, K, _ptr(scale), _ptr(a), _ptr(b), objective, _ptr(k), _stream()),
           "cq_encode_assign")
    return k


def cq_encode_scale(W: torch.Tensor, k: torch.Tensor, B: int, G: int, a, b, objective: int = CQ_FIT_CONTINUOUS) -> torch.Tensor:
    N, K = W.shape
    scale = torch.empty((N, K // G), dtype=torch.float32, device=W.device)
    _check(lib().cq_encode_scale(_ptr(W), _ptr(k), B, G, N, K, _ptr(a), _ptr(b), objective, _ptr(scale), _stream()),
           "cq_encode_scale")
    return scale


def cq_encode_losses(W: torch.Tensor, k: torch.Tensor, B: int, G: int, scale, a, b):
    """(L_C, L_A8) float64 [N, K/G] of stored codes and parameters."""
    N, K = W.shape
    lc = torch.empty((N, K // G), dtype=torch.float64, device=W.device)
    la = torch.empty_like(lc)
    _check(lib().cq_encode_losses(_ptr(W), _ptr(k), B, G, N, K, _ptr(scale), _ptr(a), _ptr(b), _ptr(lc), _ptr(la),
                                  _stream()), "cq_encode_losses")
    return lc, la


def cq_encode(W: torch.Tensor, B: int, G: int, objective: int = CQ_FIT_CONTINUOUS, effort: str = "fast"):
    """The groupwise encoder: (k int8 [N, K], scale float32, a float16, b float16 [N, K/G])."""
    N, K = W.shape
    k = torch.empty((N, K), dtype=torch.int8, device=W.device)
    scale = torch.empty((N, K // G), dtype=torch.float32, device=W.device)
    a = torch.empty((N, K // G), dtype=torch.float16, device=W.device)
    b = torch.empty_like(a)
    _check(lib().cq_encode(_ptr(W), B, G, N, K, objective, CQ_EFFORT[effort], _ptr(k), _ptr(scale), _ptr(a), _ptr(b),
                           _stream()), "cq_encode")
    return k, scale, a, b

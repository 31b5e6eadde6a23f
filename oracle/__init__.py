"""CubicQuant CPU oracle -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.

ctypes binding of ``cq_oracle.c`` (plain C, fp64, OpenMP) plus the population
distortion formulas of Section 3 in ``distortion.py``.  Only tests, the smoke
check and the CPU-baseline leg of the benchmark may import this package; the
CUDA library never does, and this package never imports the CUDA library.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "cq_oracle.c")
_LIB = os.path.join(_HERE, "libcq_oracle.so")


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (contraction off so pinned fp32 sequences hold)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared",
               "-fvisibility=hidden", "-o", _LIB + ".tmp", _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(_LIB + ".tmp", _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        L = _lib
        L.cqo_shape_margin.restype = C.c_double
        L.cqo_shape_margin.argtypes = [C.c_double, C.c_double]
        L.cqo_storage_bytes.restype = C.c_double
        L.cqo_storage_bytes.argtypes = [C.c_int64, C.c_int64, C.c_int, C.c_int]
        L.cqo_row_bytes.restype = C.c_int64
        L.cqo_row_bytes.argtypes = [C.c_int64, C.c_int]
        L.cqo_half_to_double.restype = C.c_double
        L.cqo_half_to_double.argtypes = [C.c_uint16]
        L.cqo_double_to_half.restype = C.c_uint16
        L.cqo_double_to_half.argtypes = [C.c_double]
        L.cqo_group_sse.restype = C.c_double
        L.cqo_joint_scale.restype = C.c_double
        L.cqo_gemm_a8.restype = C.c_int64
        L.cqo_num_threads.restype = C.c_int
        L.cqo_num_levels.restype = C.c_int
    return _lib


def _p(arr):
    return None if arr is None else arr.ctypes.data_as(C.c_void_p)


def _c(arr, dtype):
    arr = np.ascontiguousarray(arr, dtype=dtype)
    return arr


def _h(arr):
    """binary16 array (np.float16 or uint16 bit patterns) -> contiguous uint16 bit patterns."""
    arr = np.asarray(arr)
    if arr.dtype == np.float16:
        arr = arr.view(np.uint16)
    return np.ascontiguousarray(arr, dtype=np.uint16)


def num_threads() -> int:
    return lib().cqo_num_threads()


def num_levels(B: int) -> int:
    return lib().cqo_num_levels(B)


def shape_margin(a: float, b: float) -> float:
    return lib().cqo_shape_margin(float(a), float(b))


def storage_bytes(N, K, B, G) -> float:
    return lib().cqo_storage_bytes(N, K, B, G)


def row_bytes(K, B) -> int:
    return lib().cqo_row_bytes(K, B)


def levels(B: int, s, a16, b16) -> np.ndarray:
    """Non-negative levels of one group, fp64, length num_levels(B)."""
    out = np.zeros(num_levels(B), dtype=np.float64)
    a16 = int(_h(np.array([a16]).reshape(1))[0]) if not isinstance(a16, (int, np.integer)) else int(a16)
    b16 = int(_h(np.array([b16]).reshape(1))[0]) if not isinstance(b16, (int, np.integer)) else int(b16)
    lib().cqo_levels(C.c_int(B), C.c_float(float(s)), C.c_uint16(a16), C.c_uint16(b16), _p(out))
    return out


def levels_all(B: int, s, a, b) -> np.ndarray:
    """levels for arrays of groups: [..., num_levels(B)]."""
    s = np.asarray(s, dtype=np.float32)
    a = _h(a).reshape(-1)
    b = _h(b).reshape(-1)
    out = np.zeros((s.size, num_levels(B)), dtype=np.float64)
    sf = s.reshape(-1)
    L = lib()
    for i in range(s.size):
        L.cqo_levels(C.c_int(B), C.c_float(float(sf[i])), C.c_uint16(int(a[i])), C.c_uint16(int(b[i])),
                     C.c_void_p(out[i].ctypes.data))
    return out.reshape(s.shape + (num_levels(B),))


def carriers(B: int, a16, b16) -> np.ndarray:
    out = np.zeros(num_levels(B), dtype=np.int8)
    a16 = int(_h(np.array([a16]).reshape(1))[0]) if not isinstance(a16, (int, np.integer)) else int(a16)
    b16 = int(_h(np.array([b16]).reshape(1))[0]) if not isinstance(b16, (int, np.integer)) else int(b16)
    lib().cqo_carriers(C.c_int(B), C.c_uint16(a16), C.c_uint16(b16), _p(out))
    return out


def carriers_all(B: int, a, b) -> np.ndarray:
    a = _h(a)
    shp = a.shape
    af = a.reshape(-1)
    bf = _h(b).reshape(-1)
    out = np.zeros((af.size, num_levels(B)), dtype=np.int8)
    L = lib()
    for i in range(af.size):
        L.cqo_carriers(C.c_int(B), C.c_uint16(int(af[i])), C.c_uint16(int(bf[i])), C.c_void_p(out[i].ctypes.data))
    return out.reshape(shp + (num_levels(B),))


def pack(k: np.ndarray, B: int) -> np.ndarray:
    k = _c(k, np.int8)
    N, K = k.shape
    out = np.zeros((N, row_bytes(K, B)), dtype=np.uint8)
    lib().cqo_pack(_p(k), C.c_int64(N), C.c_int64(K), C.c_int(B), _p(out))
    return out


def unpack(codes: np.ndarray, K: int, B: int) -> np.ndarray:
    codes = _c(codes, np.uint8)
    N = codes.shape[0]
    k = np.zeros((N, K), dtype=np.int8)
    lib().cqo_unpack(_p(codes), C.c_int64(N), C.c_int64(K), C.c_int(B), _p(k))
    return k


EFFORT = {"int_absmax": 0, "int_clipped": 1, "fast": 2, "reference": 3}


def encode(W: np.ndarray, B: int, G: int, effort: str = "fast", objective: str = "continuous"):
    """Groupwise encoder: returns (k int8 [N,K], s fp32 [N,K/G], a fp16, b fp16).
    objective "continuous" minimises L_C (Section 4.1), "joint" L_C + L_A8 (Section 4.3)."""
    W = _c(W, np.float32)
    N, K = W.shape
    assert K % G == 0 and G <= 512
    ng = K // G
    k = np.zeros((N, K), dtype=np.int8)
    s = np.zeros((N, ng), dtype=np.float32)
    a = np.zeros((N, ng), dtype=np.uint16)
    b = np.zeros((N, ng), dtype=np.uint16)
    fn = {"continuous": lib().cqo_encode, "joint": lib().cqo_encode_joint}[objective]
    fn(_p(W), C.c_int64(N), C.c_int64(K), C.c_int(B), C.c_int(G), C.c_int(EFFORT[effort]), _p(k), _p(s), _p(a), _p(b))
    return k, s, a.view(np.float16), b.view(np.float16)


def joint_levels(B: int, a16, b16):
    """(z, ztilde): continuous normalised levels q(i/M) and carrier-grid levels round(127 q)/127."""
    n = num_levels(B)
    z = np.zeros(n, dtype=np.float64)
    zt = np.zeros(n, dtype=np.float64)
    a16 = int(_h(np.array([a16]))[0])
    b16 = int(_h(np.array([b16]))[0])
    lib().cqo_joint_levels(C.c_int(B), C.c_uint16(a16), C.c_uint16(b16), _p(z), _p(zt))
    return z, zt


def assign_group_joint(w, B, s, a16, b16) -> np.ndarray:
    w = _c(w, np.float32)
    k = np.zeros(w.size, dtype=np.int8)
    a16 = int(_h(np.array([a16]))[0])
    b16 = int(_h(np.array([b16]))[0])
    lib().cqo_assign_group_joint(_p(w), C.c_int(w.size), C.c_int(B), C.c_float(float(s)), C.c_uint16(a16),
                                 C.c_uint16(b16), _p(k))
    return k


def group_losses(w, B, s, a16, b16, k):
    """(L_C, L_A8) of one group for stored codes (Eq. continuous-and-carrier-loss)."""
    w = _c(w, np.float32)
    k = _c(k, np.int8)
    a16 = int(_h(np.array([a16]))[0])
    b16 = int(_h(np.array([b16]))[0])
    lc, la = C.c_double(0.0), C.c_double(0.0)
    lib().cqo_group_losses(_p(w), C.c_int(w.size), C.c_int(B), C.c_float(float(s)), C.c_uint16(a16), C.c_uint16(b16),
                           _p(k), C.byref(lc), C.byref(la))
    return lc.value, la.value


def joint_scale(w, k, B, a16, b16) -> float:
    """Scale minimising L_C + L_A8 for fixed codes and shape (Eq. carrier-aware-scale)."""
    w = _c(w, np.float32)
    k = _c(k, np.int8)
    a16 = int(_h(np.array([a16]))[0])
    b16 = int(_h(np.array([b16]))[0])
    return lib().cqo_joint_scale(_p(w), _p(k), C.c_int(w.size), C.c_int(B), C.c_uint16(a16), C.c_uint16(b16))


def assign_group(w, B, s, a16, b16) -> np.ndarray:
    w = _c(w, np.float32)
    k = np.zeros(w.size, dtype=np.int8)
    a16 = int(_h(np.array([a16]))[0])
    b16 = int(_h(np.array([b16]))[0])
    lib().cqo_assign_group(_p(w), C.c_int(w.size), C.c_int(B), C.c_float(float(s)), C.c_uint16(a16),
                           C.c_uint16(b16), _p(k))
    return k


def group_sse(w, B, s, a16, b16, k) -> float:
    w = _c(w, np.float32)
    k = _c(k, np.int8)
    a16 = int(_h(np.array([a16]))[0])
    b16 = int(_h(np.array([b16]))[0])
    return lib().cqo_group_sse(_p(w), C.c_int(w.size), C.c_int(B), C.c_float(float(s)), C.c_uint16(a16),
                               C.c_uint16(b16), _p(k))


def decode_dense(codes, s, a, b, B, G, K) -> np.ndarray:
    codes = _c(codes, np.uint8)
    s = _c(s, np.float32)
    a = _h(a)
    b = _h(b)
    N = codes.shape[0]
    out = np.zeros((N, K), dtype=np.float64)
    lib().cqo_decode_dense(_p(codes), _p(s), _p(a), _p(b), C.c_int(B), C.c_int(G), C.c_int64(N), C.c_int64(K), _p(out))
    return out


def _subset(idx):
    if idx is None:
        return None, 0
    arr = np.ascontiguousarray(idx, dtype=np.int64)
    return arr, arr.size


def gemm_model(codes, s, a, b, B, G, K, x_bf16, rows=None, cols=None, act="bf16") -> np.ndarray:
    """fp64 y[rows, cols] of the model-dtype product; x_bf16 is uint16 bit patterns [M, K] of the
    activation dtype `act` ("bf16" or "f16")."""
    codes = _c(codes, np.uint8)
    s = _c(s, np.float32)
    a = _h(a)
    b = _h(b)
    x = _c(x_bf16, np.uint16)
    N, M = codes.shape[0], x.shape[0]
    r, nr = _subset(rows)
    c, nc = _subset(cols)
    nr = nr if rows is not None else M
    nc = nc if cols is not None else N
    y = np.zeros((nr, nc), dtype=np.float64)
    lib().cqo_gemm_model_act(_p(codes), _p(s), _p(a), _p(b), C.c_int(B), C.c_int(G), C.c_int64(N), C.c_int64(K), _p(x),
                             C.c_int({"bf16": 0, "f16": 1}[act]), C.c_int64(M), _p(r), C.c_int64(nr), _p(c), C.c_int64(nc), _p(y))
    return y


def quantize_a8(x_bf16, act="bf16"):
    x = _c(x_bf16, np.uint16)
    M, K = x.shape
    x8 = np.zeros((M, K), dtype=np.int8)
    dx = np.zeros(M, dtype=np.float32)
    lib().cqo_quantize_a8_act(_p(x), C.c_int({"bf16": 0, "f16": 1}[act]), C.c_int64(M), C.c_int64(K), _p(x8), _p(dx))
    return x8, dx


def gemm_a8(codes, s, a, b, B, G, K, x8, dx, rows=None, cols=None, want_partials=False):
    """fp64 y[rows, cols] of the Dynamic-A8 product and (optionally) the int32 partials P[rows, cols, K/G]."""
    codes = _c(codes, np.uint8)
    s = _c(s, np.float32)
    a = _h(a)
    b = _h(b)
    x8 = _c(x8, np.int8)
    dx = _c(dx, np.float32)
    N, M = codes.shape[0], x8.shape[0]
    r, nr = _subset(rows)
    c, nc = _subset(cols)
    nr = nr if rows is not None else M
    nc = nc if cols is not None else N
    y = np.zeros((nr, nc), dtype=np.float64)
    P = np.zeros((nr, nc, K // G), dtype=np.int32) if want_partials else None
    bad = lib().cqo_gemm_a8(_p(codes), _p(s), _p(a), _p(b), C.c_int(B), C.c_int(G), C.c_int64(N), C.c_int64(K),
                            _p(x8), _p(dx), C.c_int64(M), _p(r), C.c_int64(nr), _p(c), C.c_int64(nc), _p(y), _p(P))
    assert bad == 0, "int32 partial bound |P_g| <= G*127^2 violated"
    return (y, P) if want_partials else y


# ----------------------------------------------------------------------------- fused MLP boundary
def silu_mul(gate: np.ndarray, up: np.ndarray) -> np.ndarray:
    """The gated activation of a SwiGLU MLP in fp64: silu(gate) * up, silu(g) = g / (1 + exp(-g))."""
    g = np.asarray(gate, np.float64)
    return g / (1.0 + np.exp(-g)) * np.asarray(up, np.float64)


def _to_bf16_bits(v: np.ndarray) -> np.ndarray:
    """fp64 -> bfloat16 bit patterns, round to nearest even (through fp32, which holds every bf16 midpoint)."""
    f = np.ascontiguousarray(v, dtype=np.float32)
    u = f.view(np.uint32)
    return ((u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)).astype(np.uint16)


def mlp_swiglu(gate_up, down, x_bf16, mode_gate_up: str = "model"):
    """The MLP boundary of Section 5.4 (last paragraph: activation and quantisation fused next to the down
    projection) as the plain composition of the operators it fuses, each with its operator-local semantics:

        h   = gate_up(x)                 model dtype or Dynamic A8, output rounded to the model dtype (bf16)
        act = bf16(silu(h[:, :I]) * h[:, I:])
        y   = down(act) in Dynamic A8    per-row absmax INT8 of act, INT8 carriers, int32 partials, fp32 rescale

    gate_up / down: dicts with codes, s, a, b, B, G, K (gate_up has 2 I output channels, down has K = I).
    Returns (y fp64 [M, N], act bf16 bits [M, I])."""
    gu, dn = gate_up, down
    if mode_gate_up == "model":
        h = gemm_model(gu["codes"], gu["s"], gu["a"], gu["b"], gu["B"], gu["G"], gu["K"], x_bf16)
    else:
        x8, dx = quantize_a8(x_bf16)
        h = gemm_a8(gu["codes"], gu["s"], gu["a"], gu["b"], gu["B"], gu["G"], gu["K"], x8, dx)
    hb = _to_bf16_bits(h)
    hv = (hb.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    inter = hv.shape[1] // 2
    act = _to_bf16_bits(silu_mul(hv[:, :inter], hv[:, inter:]))
    a8, da = quantize_a8(act)
    y = gemm_a8(dn["codes"], dn["s"], dn["a"], dn["b"], dn["B"], dn["G"], dn["K"], a8, da)
    return y, act


# ----------------------------------------------------------------------------- routed execution
def gemm_routed(experts, x_bits, route_token, expert_offset, mode: str = "model", act: str = "bf16") -> np.ndarray:
    """Routed product of Section 5.5 with routes grouped by matrix: route r (in the block of matrix e) is the
    ordinary product of token route_token[r] with matrix e.  experts: list of dicts (codes, s, a, b, B, G, K);
    returns route-major fp64 y[R, N].  Route weights and the reduction over a token's routes are not part of it."""
    x_bits = np.asarray(x_bits, np.uint16)
    route_token = np.asarray(route_token, np.int64)
    R = int(expert_offset[-1])
    N = experts[0]["codes"].shape[0]
    y = np.zeros((R, N), np.float64)
    for e, w in enumerate(experts):
        r0, r1 = int(expert_offset[e]), int(expert_offset[e + 1])
        if r1 == r0:
            continue
        xe = np.ascontiguousarray(x_bits[route_token[r0:r1]])
        if mode == "model":
            y[r0:r1] = gemm_model(w["codes"], w["s"], w["a"], w["b"], w["B"], w["G"], w["K"], xe, act=act)
        else:
            x8, dx = quantize_a8(xe, act=act)
            y[r0:r1] = gemm_a8(w["codes"], w["s"], w["a"], w["b"], w["B"], w["G"], w["K"], x8, dx)
    return y

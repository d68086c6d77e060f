"""ctypes binding of the CPU fp64 oracle (``moe_oracle.c``) -- TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the bench's CPU-baseline leg may import this
package.  It imports nothing from the CUDA package and the CUDA package imports
nothing from here.  All arrays are numpy arrays in host memory; weight tensors
are passed as raw bytes (uint8/uint16/float32 arrays) in the layouts the C file
documents.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "moe_oracle.c")
_LIB = os.path.join(_HERE, "libmoe_oracle.so")

W_FP32, W_BF16, W_FP8E4M3_B128, W_MXFP4 = 0, 1, 2, 3
FFN_SWIGLU, FFN_GPTOSS = 0, 1
ACT_FP32, ACT_BF16 = 0, 1
SCORE_SOFTMAX, SCORE_SIGMOID = 0, 1


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (``-O2 -fopenmp``); returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


class _Cfg(C.Structure):
    _fields_ = [("H", C.c_int32), ("I", C.c_int32), ("E", C.c_int32), ("top_k", C.c_int32),
                ("n_shared", C.c_int32), ("wfmt", C.c_int32), ("afmt", C.c_int32),
                ("score", C.c_int32), ("routed_scale", C.c_double), ("ffn_kind", C.c_int32),
                ("n_group", C.c_int32), ("topk_group", C.c_int32), ("act_quant", C.c_int32)]


class _Layer(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in (
        "router_w", "w_gate", "w_up", "w_down", "s_gate", "s_up", "s_down",
        "sh_gate", "sh_up", "sh_down", "sh_s_gate", "sh_s_up", "sh_s_down", "b_gate", "b_up", "b_down", "router_bias")]


@dataclass
class Config:
    H: int
    I: int
    E: int
    top_k: int
    n_shared: int = 0
    wfmt: int = W_FP32
    afmt: int = ACT_FP32
    score: int = SCORE_SOFTMAX
    routed_scale: float = 1.0
    ffn_kind: int = 0   # 0 bias-free SwiGLU; 1 GPT-OSS form (clamped, biased; layer keys b_gate / b_up / b_down)
    n_group: int = 0    # > 0: DeepSeek group-limited routing (sigmoid scores; layer key router_bias)
    topk_group: int = 0
    act_quant: int = 0  # 1 / 2: FP8 activations with 1x128 scales (binary32 / power-of-two scales) in front of both expert GEMMs

    def c(self) -> _Cfg:
        return _Cfg(self.H, self.I, self.E, self.top_k, self.n_shared, self.wfmt, self.afmt,
                    self.score, self.routed_scale, self.ffn_kind, self.n_group, self.topk_group, self.act_quant)


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.oracle_decode_bf16.restype = C.c_double
        _lib.oracle_decode_bf16.argtypes = [C.c_uint16]
        _lib.oracle_decode_e4m3.restype = C.c_double
        _lib.oracle_decode_e4m3.argtypes = [C.c_uint8]
        _lib.oracle_encode_e4m3.restype = C.c_uint8
        _lib.oracle_encode_e4m3.argtypes = [C.c_float]
        _lib.oracle_decode_e2m1.restype = C.c_double
        _lib.oracle_decode_e2m1.argtypes = [C.c_uint8]
        _lib.oracle_decode_e8m0.restype = C.c_double
        _lib.oracle_decode_e8m0.argtypes = [C.c_uint8]
        _lib.oracle_expert_code_bytes.restype = C.c_int64
        _lib.oracle_expert_scale_bytes.restype = C.c_int64
        _lib.oracle_union_perm.restype = C.c_int32
        _lib.oracle_moe_verify.restype = C.c_int32
        _lib.oracle_moe_dense.restype = C.c_int32
        _lib.oracle_num_threads.restype = C.c_int32
        _lib.oracle_select_drafts.restype = C.c_int32
    return _lib


def _p(a):
    if a is None:
        return None
    assert isinstance(a, np.ndarray) and a.flags["C_CONTIGUOUS"], "need contiguous numpy arrays"
    return C.c_void_p(a.ctypes.data)


def _layer(layer: dict) -> _Layer:
    """``layer`` maps the field names of the C struct to numpy arrays (missing = NULL)."""
    L = _Layer()
    for name, _ in _Layer._fields_:
        a = layer.get(name)
        setattr(L, name, None if a is None else a.ctypes.data)
    return L


def decode_bf16(b: int) -> float:
    return lib().oracle_decode_bf16(b)


def decode_e4m3(b: int) -> float:
    return lib().oracle_decode_e4m3(b)


def encode_e4m3(f: float) -> int:
    return lib().oracle_encode_e4m3(f)


def act_quant(x: np.ndarray, mode: int = 1):
    """FP8 1x128 quantisation of the rows of x (float32 [..., n]): (codes uint8 [..., n],
    scales float32 [..., ceil(n / 128)])."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    n = x.shape[-1]
    rows = x.reshape(-1, n)
    codes = np.zeros(rows.shape, dtype=np.uint8)
    scales = np.zeros((rows.shape[0], (n + 127) // 128), dtype=np.float32)
    for r in range(rows.shape[0]):
        lib().oracle_act_quant(C.c_void_p(rows[r].ctypes.data), C.c_int64(n), C.c_int32(mode),
                               C.c_void_p(codes[r].ctypes.data), C.c_void_p(scales[r].ctypes.data))
    return codes.reshape(x.shape), scales.reshape(x.shape[:-1] + (scales.shape[1],))


def decode_e2m1(b: int) -> float:
    return lib().oracle_decode_e2m1(b)


def decode_e8m0(b: int) -> float:
    return lib().oracle_decode_e8m0(b)


def expert_code_bytes(cfg: Config) -> int:
    c = cfg.c()
    return lib().oracle_expert_code_bytes(C.byref(c))


def expert_scale_bytes(cfg: Config) -> int:
    c = cfg.c()
    return lib().oracle_expert_scale_bytes(C.byref(c))


def num_threads() -> int:
    return lib().oracle_num_threads()


def decode_weight_row(wfmt: int, w: np.ndarray, s, e: int, N: int, K: int, n: int) -> np.ndarray:
    out = np.empty(K, dtype=np.float64)
    lib().oracle_decode_weight_row(C.c_int32(wfmt), _p(w), _p(s), C.c_int64(e), C.c_int64(N),
                                   C.c_int64(K), C.c_int64(n), _p(out))
    return out


def router_logits(cfg: Config, x: np.ndarray, router_w: np.ndarray, gamma: int) -> np.ndarray:
    out = np.empty((gamma, cfg.E), dtype=np.float64)
    c = cfg.c()
    assert router_w.dtype == np.float32
    lib().oracle_router_logits(C.byref(c), _p(x), _p(router_w), C.c_int32(gamma), _p(out))
    return out


def topk(cfg: Config, logits: np.ndarray):
    gamma = logits.shape[0]
    logits = np.ascontiguousarray(logits, dtype=np.float64)
    ids = np.empty((gamma, cfg.top_k), dtype=np.int32)
    w = np.empty((gamma, cfg.top_k), dtype=np.float64)
    gap = np.empty(gamma, dtype=np.float64)
    c = cfg.c()
    lib().oracle_topk(C.byref(c), _p(logits), C.c_int32(gamma), _p(ids), _p(w), _p(gap))
    return ids, w, gap


def topk_grouped(cfg: Config, logits: np.ndarray, bias=None):
    gamma = logits.shape[0]
    logits = np.ascontiguousarray(logits, dtype=np.float64)
    if bias is not None:
        bias = np.ascontiguousarray(bias, dtype=np.float32)
    ids = np.empty((gamma, cfg.top_k), dtype=np.int32)
    w = np.empty((gamma, cfg.top_k), dtype=np.float64)
    gap = np.empty(gamma, dtype=np.float64)
    c = cfg.c()
    lib().oracle_topk_grouped(C.byref(c), _p(logits), _p(bias), C.c_int32(gamma), _p(ids), _p(w), _p(gap))
    return ids, w, gap


def union_perm(E: int, k: int, ids: np.ndarray):
    ids = np.ascontiguousarray(ids, dtype=np.int32)
    gamma = ids.shape[0]
    A = gamma * k
    union_ids = np.full(E, -1, dtype=np.int32)
    offsets = np.full(E + 1, -1, dtype=np.int32)
    perm = np.empty(A, dtype=np.int32)
    inv = np.empty(A, dtype=np.int32)
    U = lib().oracle_union_perm(C.c_int32(E), C.c_int32(k), C.c_int32(gamma), _p(ids),
                                _p(union_ids), _p(offsets), _p(perm), _p(inv))
    return U, union_ids[:U].copy(), offsets[:U + 1].copy(), perm, inv


def expert_ffn(cfg: Config, layer: dict, e: int, xs: np.ndarray, shared: bool = False) -> np.ndarray:
    xs = np.ascontiguousarray(xs, dtype=np.float64)
    m = xs.shape[0]
    out = np.empty((m, cfg.H), dtype=np.float64)
    c, L = cfg.c(), _layer(layer)
    lib().oracle_expert_ffn(C.byref(c), C.byref(L), C.c_int32(int(shared)), C.c_int32(e),
                            C.c_int32(m), _p(xs), _p(out))
    return out


@dataclass
class Result:
    n_active: int
    y: np.ndarray | None
    topk_ids: np.ndarray
    topk_w: np.ndarray
    union_ids: np.ndarray
    offsets: np.ndarray
    perm: np.ndarray
    inv_perm: np.ndarray
    gap: np.ndarray
    logits: np.ndarray


def moe_verify(cfg: Config, layer: dict, x: np.ndarray, gamma: int, override_w=None,
               skip_ffn: bool = False) -> Result:
    """Run the whole layer over ``gamma`` tokens; ``y`` is float64 [gamma, H]."""
    k, E = cfg.top_k, cfg.E
    A = gamma * k
    y = None if skip_ffn else np.empty((gamma, cfg.H), dtype=np.float64)
    ids = np.empty((gamma, k), dtype=np.int32)
    w = np.empty((gamma, k), dtype=np.float64)
    union_ids = np.full(E, -1, dtype=np.int32)
    offsets = np.full(E + 1, -1, dtype=np.int32)
    perm = np.empty(A, dtype=np.int32)
    inv = np.empty(A, dtype=np.int32)
    gap = np.empty(gamma, dtype=np.float64)
    logits = np.empty((gamma, E), dtype=np.float64)
    if override_w is not None:
        override_w = np.ascontiguousarray(override_w, dtype=np.float64)
        assert override_w.size == A
    c, L = cfg.c(), _layer(layer)
    U = lib().oracle_moe_verify(C.byref(c), C.byref(L), _p(x), C.c_int32(gamma), _p(override_w),
                                C.c_int32(int(skip_ffn)), _p(y), _p(ids), _p(w), _p(union_ids),
                                _p(offsets), _p(perm), _p(inv), _p(gap), _p(logits))
    if U < 0:
        raise ValueError("oracle_moe_verify: bad arguments")
    return Result(U, y, ids, w, union_ids[:U].copy(), offsets[:U + 1].copy(), perm, inv, gap,
                  logits)


def moe_dense(cfg: Config, layer: dict, x: np.ndarray, gamma: int) -> np.ndarray:
    y = np.empty((gamma, cfg.H), dtype=np.float64)
    c, L = cfg.c(), _layer(layer)
    rc = lib().oracle_moe_dense(C.byref(c), C.byref(L), _p(x), C.c_int32(gamma), _p(y))
    if rc != 0:
        raise ValueError("oracle_moe_dense: bad arguments")
    return y


def select_drafts(parent, P, pred, gamma: int, eps: float = 1e-6, buffer0=None, global_cost: bool = False):
    """Algorithm 1 on a draft tree.  pred: uint32 [n, W] bitmaps.  Returns (selected, costs, buffer)."""
    parent = np.ascontiguousarray(parent, dtype=np.int32)
    P = np.ascontiguousarray(P, dtype=np.float32)
    pred = np.ascontiguousarray(pred, dtype=np.uint32)
    n, W = pred.shape
    if buffer0 is not None:
        buffer0 = np.ascontiguousarray(buffer0, dtype=np.uint32)
    sel = np.full(gamma, -1, dtype=np.int32)
    costs = np.zeros(gamma, dtype=np.int32)
    buf = np.zeros(W, dtype=np.uint32)
    cnt = lib().oracle_select_drafts(C.c_int32(n), C.c_int32(W), _p(parent), _p(P), _p(pred), _p(buffer0),
                                     C.c_int32(gamma), C.c_float(eps), C.c_int32(int(global_cost)), _p(sel),
                                     _p(costs), _p(buf))
    if cnt < 0:
        raise ValueError("oracle_select_drafts: bad arguments")
    return sel[:cnt].copy(), costs[:cnt].copy(), buf

"""ctypes binding with the same names as the C ABI (see include/moev.h)."""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libmoev.so")

W_FP32, W_BF16, W_FP8E4M3_B128, W_MXFP4 = 0, 1, 2, 3
ACT_FP32, ACT_BF16 = 0, 1
SCORE_SOFTMAX, SCORE_SIGMOID = 0, 1
IMPL_AUTO, IMPL_SIMT, IMPL_TCGEN05 = 0, 1, 2
STATUS = {0: "MOEV_OK", 1: "MOEV_EINVAL", 2: "MOEV_EUNSUPPORTED", 3: "MOEV_ECUDA",
          4: "MOEV_ENOMEM", 5: "MOEV_ETIMEOUT"}

EXPORTS = ("moev_create", "moev_destroy", "moev_verify", "moev_verify_host", "moev_status_sync",
           "moev_last_error", "moev_expert_bytes", "moev_expert_code_bytes",
           "moev_launches_per_call", "moev_resolved_impl", "moev_profile_enable",
           "moev_profile_read", "moev_route_topk_static", "moev_route_topk_static_scratch_floats", "moev_select_drafts",
           "moev_verify_pipeline", "moev_prefetch_enable", "moev_verify_chain", "moev_ffn_span_enable",
           "moev_ffn_span_read")


class MoevError(RuntimeError):
    def __init__(self, status: int, text: str = ""):
        self.status = status
        super().__init__(f"{STATUS.get(status, status)}: {text}")


FFN_SWIGLU, FFN_GPTOSS = 0, 1
ACTQ_NONE, ACTQ_FP8_B128, ACTQ_FP8_B128_POW2 = 0, 1, 2


class _Config(C.Structure):
    _fields_ = [("H", C.c_int32), ("I", C.c_int32), ("E", C.c_int32), ("top_k", C.c_int32),
                ("n_shared", C.c_int32), ("max_tokens", C.c_int32), ("wfmt", C.c_int32),
                ("afmt", C.c_int32), ("score", C.c_int32), ("impl", C.c_int32),
                ("routed_scale", C.c_float), ("ffn_kind", C.c_int32), ("n_group", C.c_int32),
                ("topk_group", C.c_int32), ("act_quant", C.c_int32)]


_LAYER_FIELDS = ("router_w", "w_gate", "w_up", "w_down", "s_gate", "s_up", "s_down",
                 "sh_gate", "sh_up", "sh_down", "sh_s_gate", "sh_s_up", "sh_s_down", "b_gate", "b_up", "b_down", "router_bias")
_OUT_FIELDS = ("y", "topk_ids", "topk_w", "union_ids", "offsets", "perm", "n_active")


class _Layer(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in _LAYER_FIELDS] + [("predicted_ids", C.c_void_p), ("n_predicted", C.c_int32)]


class _Out(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in _OUT_FIELDS]


@dataclass
class MoevConfig:
    H: int
    I: int
    E: int
    top_k: int
    n_shared: int = 0
    max_tokens: int = 128
    wfmt: int = W_BF16
    afmt: int = ACT_BF16
    score: int = SCORE_SOFTMAX
    impl: int = IMPL_AUTO
    routed_scale: float = 1.0
    ffn_kind: int = 0   # FFN_SWIGLU; FFN_GPTOSS = clamped, biased GPT-OSS expert (layer keys b_gate / b_up / b_down)
    n_group: int = 0    # > 0: DeepSeek group-limited routing (sigmoid scores; layer key router_bias)
    topk_group: int = 0
    act_quant: int = 0  # ACTQ_FP8_B128 / ACTQ_FP8_B128_POW2: FP8 activations with 1x128 scales in front of both expert GEMMs

    def c(self) -> _Config:
        return _Config(self.H, self.I, self.E, self.top_k, self.n_shared, self.max_tokens,
                       self.wfmt, self.afmt, self.score, self.impl, self.routed_scale, self.ffn_kind,
                       self.n_group, self.topk_group, self.act_quant)


_lib = None


def lib_path() -> str:
    return _LIB_PATH


def lib() -> C.CDLL:
    """Load libmoev.so; raises (never falls back) when it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise ImportError(f"{_LIB_PATH} not found: build it with "
                              "`python -m paper_2607_12696_b200.build` (there is no CPU fallback)")
        L = C.CDLL(_LIB_PATH)
        L.moev_create.restype = C.c_int
        L.moev_create.argtypes = [C.POINTER(_Config), C.POINTER(C.c_void_p)]
        L.moev_destroy.restype = C.c_int
        L.moev_destroy.argtypes = [C.c_void_p]
        L.moev_verify.restype = C.c_int
        L.moev_verify.argtypes = [C.c_void_p, C.POINTER(_Layer), C.c_void_p, C.c_int32,
                                  C.POINTER(_Out), C.c_void_p]
        L.moev_verify_pipeline.restype = C.c_int
        L.moev_verify_pipeline.argtypes = [C.c_void_p, C.c_int32, C.POINTER(_Layer), C.POINTER(C.c_void_p), C.c_int32,
                                           C.POINTER(_Out), C.c_void_p]
        L.moev_verify_chain.restype = C.c_int
        L.moev_verify_chain.argtypes = [C.c_void_p, C.c_int32, C.POINTER(_Layer), C.c_void_p, C.c_int32,
                                        C.POINTER(_Out), C.c_void_p]
        L.moev_verify_host.restype = C.c_int
        L.moev_verify_host.argtypes = [C.c_void_p, C.POINTER(_Layer), C.c_void_p, C.c_int32,
                                       C.c_void_p, C.c_void_p, C.c_void_p]
        L.moev_status_sync.restype = C.c_int
        L.moev_status_sync.argtypes = [C.c_void_p, C.c_void_p]
        L.moev_last_error.restype = C.c_char_p
        L.moev_last_error.argtypes = [C.c_void_p]
        L.moev_expert_bytes.restype = C.c_size_t
        L.moev_expert_bytes.argtypes = [C.POINTER(_Config)]
        L.moev_expert_code_bytes.restype = C.c_size_t
        L.moev_expert_code_bytes.argtypes = [C.POINTER(_Config)]
        L.moev_launches_per_call.restype = C.c_int32
        L.moev_launches_per_call.argtypes = [C.c_void_p]
        L.moev_resolved_impl.restype = C.c_int32
        L.moev_resolved_impl.argtypes = [C.c_void_p]
        L.moev_profile_enable.restype = C.c_int
        L.moev_profile_enable.argtypes = [C.c_void_p, C.c_int32]
        L.moev_prefetch_enable.restype = C.c_int
        L.moev_prefetch_enable.argtypes = [C.c_void_p, C.c_int32]
        L.moev_profile_read.restype = C.c_int
        L.moev_profile_read.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(C.c_double),
                                        C.POINTER(C.c_int32)]
        L.moev_ffn_span_enable.restype = C.c_int
        L.moev_ffn_span_enable.argtypes = [C.c_void_p, C.c_int32]
        L.moev_ffn_span_read.restype = C.c_int
        L.moev_ffn_span_read.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(C.c_double)]
        L.moev_route_topk_static.restype = C.c_int
        L.moev_route_topk_static.argtypes = [C.POINTER(_Config), C.c_void_p, C.c_void_p, C.c_int32,
                                             C.c_void_p, C.c_void_p, C.c_void_p]
        L.moev_route_topk_static_scratch_floats.restype = C.c_size_t
        L.moev_route_topk_static_scratch_floats.argtypes = [C.c_int32, C.c_int32, C.c_int32]
        L.moev_select_drafts.restype = C.c_int
        L.moev_select_drafts.argtypes = [C.c_int32, C.c_int32] + [C.c_void_p] * 4 + [C.c_int32, C.c_float, C.c_int32] + \
                                        [C.c_void_p] * 6
        _lib = L
    return _lib


def expert_bytes(cfg: MoevConfig) -> int:
    c = cfg.c()
    return lib().moev_expert_bytes(C.byref(c))


def expert_code_bytes(cfg: MoevConfig) -> int:
    c = cfg.c()
    return lib().moev_expert_code_bytes(C.byref(c))


def route_topk_static(cfg: MoevConfig, router_w: torch.Tensor, x: torch.Tensor, gamma: int,
                      topk_ids: torch.Tensor, topk_w: torch.Tensor):
    """moev_route_topk_static: router top-k for callers that may not allocate device memory.

    Needs no context; the scratch is the fixed array inside the library, shared by all calls
    (do not overlap calls on the GPU).  Asynchronous on torch's current stream."""
    c = cfg.c()
    st = lib().moev_route_topk_static(C.byref(c), router_w.data_ptr(), x.data_ptr(), gamma,
                                      topk_ids.data_ptr(), topk_w.data_ptr(),
                                      C.c_void_p(torch.cuda.current_stream().cuda_stream))
    if st != 0:
        raise MoevError(st, "moev_route_topk_static rejected the call (arguments, or the problem "
                            "exceeds the fixed scratch array)")


def select_drafts(parent: torch.Tensor, P: torch.Tensor, pred: torch.Tensor, gamma: int, eps: float = 1e-6,
                  buffer0: torch.Tensor = None, global_cost: bool = False, out: tuple = None):
    """moev_select_drafts: Algorithm 1 on device tensors (parent int32 [n], P float32 [n], pred
    int32/uint32 bitmaps [n, W]).  Returns device tensors (selected [gamma], costs [gamma],
    buffer [W], n_selected [1], workspace [n * W + 516]); asynchronous on the current stream.  Pass the
    tuple a previous call returned as ``out`` to reuse its tensors (no allocation)."""
    n, W = pred.shape
    dev = pred.device
    if out is None:
        out = (torch.full((gamma,), -1, dtype=torch.int32, device=dev),
               torch.zeros(gamma, dtype=torch.int32, device=dev),
               torch.zeros(W, dtype=torch.int32, device=dev),
               torch.zeros(1, dtype=torch.int32, device=dev),
               torch.empty(n * W + 516, dtype=torch.int32, device=dev))
    selected, costs, buf, nsel, traj = out
    st = lib().moev_select_drafts(n, W, parent.data_ptr(), P.data_ptr(), pred.data_ptr(), _ptr(buffer0), gamma,
                                  eps, int(global_cost), traj.data_ptr(), selected.data_ptr(), costs.data_ptr(),
                                  buf.data_ptr(), nsel.data_ptr(), C.c_void_p(torch.cuda.current_stream().cuda_stream))
    if st != 0:
        raise MoevError(st, "moev_select_drafts rejected the call")
    return out


def static_scratch_floats(H: int, E: int, gamma: int) -> int:
    return lib().moev_route_topk_static_scratch_floats(H, E, gamma)


def _ptr(t):
    return None if t is None else t.data_ptr()


def make_layer(tensors: dict) -> _Layer:
    """Pack device tensors (keys = moev_layer field names; missing/None = NULL)."""
    L = _Layer()
    for n in _LAYER_FIELDS:
        t = tensors.get(n)
        if t is not None:
            assert t.is_cuda and t.is_contiguous(), f"{n} must be a contiguous CUDA tensor"
        setattr(L, n, _ptr(t))
    pred = tensors.get("predicted_ids")
    if pred is not None:
        assert pred.is_cuda and pred.dtype == torch.int32 and pred.is_contiguous()
        L.predicted_ids, L.n_predicted = pred.data_ptr(), pred.numel()
    return L


class MoeVerifier:
    """Owns one ``moev_ctx``.  ``verify`` enqueues on torch's current stream."""

    def __init__(self, cfg: MoevConfig):
        self.cfg = cfg
        self._h = C.c_void_p()
        c = cfg.c()
        st = lib().moev_create(C.byref(c), C.byref(self._h))
        if st != 0:
            self._h = None
            raise MoevError(st, "moev_create failed")

    def close(self):
        if getattr(self, "_h", None):
            lib().moev_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, st: int):
        if st != 0:
            raise MoevError(st, lib().moev_last_error(self._h).decode())

    @staticmethod
    def _stream():
        return C.c_void_p(torch.cuda.current_stream().cuda_stream)

    def alloc_out(self, gamma: int, diagnostics: bool = True) -> dict:
        cfg, dev = self.cfg, "cuda"
        out = {"y": torch.empty(gamma, cfg.H, device=dev,
                                dtype=torch.float32 if cfg.afmt == ACT_FP32 else torch.bfloat16),
               "n_active": torch.zeros(1, dtype=torch.int32, device=dev)}
        if diagnostics:
            out.update(topk_ids=torch.full((gamma, cfg.top_k), -1, dtype=torch.int32, device=dev),
                       topk_w=torch.zeros(gamma, cfg.top_k, dtype=torch.float32, device=dev),
                       union_ids=torch.full((cfg.E,), -1, dtype=torch.int32, device=dev),
                       offsets=torch.full((cfg.E + 1,), -1, dtype=torch.int32, device=dev),
                       perm=torch.full((gamma * cfg.top_k,), -1, dtype=torch.int32, device=dev))
        return out

    def verify(self, layer: _Layer, x: torch.Tensor, gamma: int, out: dict):
        """moev_verify: asynchronous on the current stream; ``out`` maps moev_out fields to tensors."""
        O = _Out()
        for n in _OUT_FIELDS:
            setattr(O, n, _ptr(out.get(n)))
        self._check(lib().moev_verify(self._h, C.byref(layer), _ptr(x), gamma, C.byref(O),
                                      self._stream()))

    def verify_pipeline(self, layers: list, xs: list, gamma: int, outs: list):
        """moev_verify_pipeline: independent layers back to back, the router of each overlapping
        the tail of the previous layer's expert kernel."""
        n = len(layers)
        assert len(xs) == n and len(outs) == n
        LA = (_Layer * n)(*layers)
        XA = (C.c_void_p * n)(*[x.data_ptr() for x in xs])
        OA = (_Out * n)()
        for i, out in enumerate(outs):
            for f in _OUT_FIELDS:
                setattr(OA[i], f, _ptr(out.get(f)))
        self._check(lib().moev_verify_pipeline(self._h, n, LA, XA, gamma, OA, self._stream()))

    def verify_chain(self, layers: list, x0: torch.Tensor, gamma: int, outs: list):
        """moev_verify_chain: dependent layers, outs[l]["y"] is the input of layer l + 1."""
        n = len(layers)
        assert len(outs) == n
        LA = (_Layer * n)(*layers)
        OA = (_Out * n)()
        for i, out in enumerate(outs):
            for f in _OUT_FIELDS:
                setattr(OA[i], f, _ptr(out.get(f)))
        self._check(lib().moev_verify_chain(self._h, n, LA, _ptr(x0), gamma, OA, self._stream()))

    def verify_host(self, layer: _Layer, x_host: torch.Tensor, gamma: int, y_host: torch.Tensor,
                    n_active_host: torch.Tensor):
        """moev_verify_host: host x in, host y / n_active out (synchronous)."""
        assert not x_host.is_cuda and not y_host.is_cuda and not n_active_host.is_cuda
        self._check(lib().moev_verify_host(self._h, C.byref(layer), x_host.data_ptr(), gamma,
                                           y_host.data_ptr(), n_active_host.data_ptr(),
                                           self._stream()))

    def status_sync(self):
        self._check(lib().moev_status_sync(self._h, self._stream()))

    def launches_per_call(self) -> int:
        return lib().moev_launches_per_call(self._h)

    def resolved_impl(self) -> int:
        return lib().moev_resolved_impl(self._h)

    def prefetch_enable(self, on: bool):
        """moev_prefetch_enable: L2 prefetch of shared / predicted experts' weights during routing."""
        self._check(lib().moev_prefetch_enable(self._h, int(on)))

    def profile_enable(self, on: bool):
        self._check(lib().moev_profile_enable(self._h, int(on)))

    def ffn_span_enable(self, on: bool):
        self._check(lib().moev_ffn_span_enable(self._h, int(on)))

    def ffn_span_read(self) -> float:
        us = C.c_double()
        self._check(lib().moev_ffn_span_read(self._h, self._stream(), C.byref(us)))
        return us.value

    def profile_read(self):
        us = (C.c_double * 6)()
        n = C.c_int32()
        self._check(lib().moev_profile_read(self._h, self._stream(), us, C.byref(n)))
        return [us[i] for i in range(6)], n.value

"""Test helpers: library-only (torch) decoding of the raw weight formats and a dense
float64 evaluation of the layer built from library routines.  Independent of both the
oracle's C code and the CUDA path."""
from __future__ import annotations

import numpy as np
import torch
import torch.nn.functional as F

import synth


def torch_decode(shape: synth.Shape, w: torch.Tensor, s) -> torch.Tensor:
    """[n,N,K(raw)] raw weights -> float64 [n,N,K] using torch's own dtype casts."""
    w = w.cpu()
    if shape.wfmt == synth.W_FP32:
        return w.to(torch.float64)
    if shape.wfmt == synth.W_BF16:
        return w.to(torch.float64)
    if shape.wfmt == synth.W_FP8E4M3_B128:
        v = w.view(torch.float8_e4m3fn).to(torch.float64)
        n, N, K = v.shape
        sc = s.cpu().to(torch.float64)
        sc = sc.repeat_interleave(128, dim=1)[:, :N].repeat_interleave(128, dim=2)[:, :, :K]
        return v * sc
    # mxfp4: unpack nibbles with integer ops, magnitudes from the OCP e2m1 value table
    table = torch.tensor([0, .5, 1, 1.5, 2, 3, 4, 6, -0., -.5, -1, -1.5, -2, -3, -4, -6],
                         dtype=torch.float64)
    lo = (w & 15).long()
    hi = (w >> 4).long()
    codes = torch.stack([lo, hi], dim=-1).flatten(-2)
    v = table[codes]
    sc = s.cpu().view(torch.float8_e8m0fnu).to(torch.float64).repeat_interleave(32, dim=2)
    return v * sc


def dense_weights(shape: synth.Shape, weights: dict) -> dict:
    out = {}
    for name in ("gate", "up", "down"):
        out[name] = torch_decode(shape, weights["w_" + name], weights["s_" + name])
        if shape.n_shared:
            out["sh_" + name] = torch_decode(shape, weights["sh_" + name], weights["sh_s_" + name])
    return out


def torch_ffn(dw: dict, e: int, x: torch.Tensor, prefix: str = "") -> torch.Tensor:
    g = x @ dw[prefix + "gate"][e].T
    p = x @ dw[prefix + "up"][e].T
    return (F.silu(g) * p) @ dw[prefix + "down"][e].T


def torch_dense_layer(shape: synth.Shape, router_w: torch.Tensor, weights: dict,
                      x: torch.Tensor) -> torch.Tensor:
    """Dense float64 MoE layer from library ops (matmul, topk, softmax/sigmoid, silu);
    only valid when the top-k decision has no exact ties."""
    dw = dense_weights(shape, weights)
    xd = x.cpu().to(torch.float64)
    logits = xd @ router_w.cpu().to(torch.float64).T
    top, ids = torch.topk(logits, shape.top_k, dim=1)
    if shape.score == synth.SCORE_SOFTMAX:
        full = torch.softmax(logits, dim=1).gather(1, ids)
        w = full / full.sum(dim=1, keepdim=True)
    else:
        sg = torch.sigmoid(top)
        w = shape.routed_scale * sg / sg.sum(dim=1, keepdim=True)
    y = torch.zeros(xd.shape[0], shape.H, dtype=torch.float64)
    for e in range(shape.E):
        gate = torch.zeros(xd.shape[0], dtype=torch.float64)
        for j in range(shape.top_k):
            gate = gate + torch.where(ids[:, j] == e, w[:, j], torch.zeros_like(w[:, j]))
        if gate.abs().sum() == 0:
            continue
        y += gate[:, None] * torch_ffn(dw, e, xd)
    for s_ in range(shape.n_shared):
        y += torch_ffn(dw, s_, xd, "sh_")
    return y


def rel_err(y: np.ndarray, ref: np.ndarray) -> float:
    """max over tokens of max_i |y - ref| / max_i |ref| (the output-parity metric)."""
    y = np.asarray(y, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    num = np.abs(y - ref).max(axis=1)
    den = np.abs(ref).max(axis=1)
    den = np.where(den == 0, 1.0, den)
    return float((num / den).max())


def small_shape(base: str, **kw) -> synth.Shape:
    """A reduced copy of a model-shaped config (same formats/scoring, smaller dims)."""
    return synth.SHAPES[base].scaled(**kw)

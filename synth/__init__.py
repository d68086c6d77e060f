"""Seeded synthetic inputs for the MoE verification layer.

This module only *draws and encodes inputs* (shapes, value distributions,
routing structure); it contains none of the layer's arithmetic and is the one
module both the CPU oracle's tests and the CUDA path's tests / bench may use.
Everything is a ``torch`` tensor of raw storage types (float32, bfloat16 viewed
as int16 where needed, uint8 codes) on the requested device.

Shapes follow Table 13 of the paper (experts per layer, top-k, shared expert)
and the workload list of the benchmark definition:

=========  =====  =====  ====  ==  =======  ==========  =======  =======
name       H      I      E     k   shared   weights     act      score
=========  =====  =====  ====  ==  =======  ==========  =======  =======
tiny       256    128    16    2   0        fp32        fp32     softmax
qwen       4096   1536   128   8   0        bf16        bf16     softmax
deepseek   7168   2048   256   8   1        fp8 b128    bf16     sigmoid
gptoss     2880   2880   128   4   0        mxfp4       bf16     softmax
=========  =====  =====  ====  ==  =======  ==========  =======  =======
"""
from __future__ import annotations

import hashlib
from dataclasses import dataclass, replace

import numpy as np
import torch

MASTER_SEED = 260712696

W_FP32, W_BF16, W_FP8E4M3_B128, W_MXFP4 = 0, 1, 2, 3
ACT_FP32, ACT_BF16 = 0, 1
SCORE_SOFTMAX, SCORE_SIGMOID = 0, 1


@dataclass(frozen=True)
class Shape:
    name: str
    H: int
    I: int
    E: int
    top_k: int
    n_shared: int
    wfmt: int
    afmt: int
    score: int
    routed_scale: float = 1.0

    def scaled(self, **kw) -> "Shape":
        return replace(self, **kw)

    def code_bytes_per_expert(self) -> int:
        el = 3 * self.H * self.I
        return {W_FP32: el * 4, W_BF16: el * 2, W_FP8E4M3_B128: el, W_MXFP4: el // 2}[self.wfmt]

    def scale_bytes_per_expert(self) -> int:
        if self.wfmt == W_FP8E4M3_B128:
            return 3 * _cdiv(self.H, 128) * _cdiv(self.I, 128) * 4
        if self.wfmt == W_MXFP4:
            return 3 * self.H * self.I // 32
        return 0

    def bytes_per_expert(self) -> int:
        return self.code_bytes_per_expert() + self.scale_bytes_per_expert()


SHAPES = {
    "tiny": Shape("tiny", 256, 128, 16, 2, 0, W_FP32, ACT_FP32, SCORE_SOFTMAX),
    "qwen": Shape("qwen", 4096, 1536, 128, 8, 0, W_BF16, ACT_BF16, SCORE_SOFTMAX),
    "deepseek": Shape("deepseek", 7168, 2048, 256, 8, 1, W_FP8E4M3_B128, ACT_BF16, SCORE_SIGMOID),
    "gptoss": Shape("gptoss", 2880, 2880, 128, 4, 0, W_MXFP4, ACT_BF16, SCORE_SOFTMAX),
}


def _cdiv(a: int, b: int) -> int:
    return (a + b - 1) // b


def stream_seed(*parts) -> int:
    """Per-tensor seed: hash of (master seed, config id, layer, tensor name, ...)."""
    h = hashlib.sha256(("/".join(str(p) for p in (MASTER_SEED,) + parts)).encode()).digest()
    return int.from_bytes(h[:8], "little") & ((1 << 62) - 1)


def _gen(device, *parts) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(stream_seed(*parts))
    return g


# ----------------------------------------------------------------- encoders

_E2M1_MAGS = (0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0)
# decision boundaries between neighbouring e2m1 magnitudes (midpoints)
_E2M1_MID = (0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0)


def encode_fp8_b128(w: torch.Tensor):
    """w [N,K] float32 -> (codes uint8 [N,K], scales float32 [ceil(N/128), ceil(K/128)]).

    scale = amax(block)/448, code = round-to-nearest e4m3 of w/scale (torch's cast)."""
    N, K = w.shape
    nb, kb = _cdiv(N, 128), _cdiv(K, 128)
    wp = torch.zeros(nb * 128, kb * 128, dtype=torch.float32, device=w.device)
    wp[:N, :K] = w
    blk = wp.view(nb, 128, kb, 128)
    amax = blk.abs().amax(dim=(1, 3)).clamp_min(1e-12)
    s = (amax / 448.0).to(torch.float32)
    q = (blk / s.view(nb, 1, kb, 1)).clamp(-448.0, 448.0).to(torch.float8_e4m3fn)
    codes = q.view(torch.uint8).view(nb * 128, kb * 128)[:N, :K].contiguous()
    return codes, s.contiguous()


def encode_mxfp4(w: torch.Tensor):
    """w [N,K] float32 (K % 32 == 0) -> (packed uint8 [N,K/2], e8m0 scales uint8 [N,K/32]).

    Per 32 along K: scale 2^ceil(log2(amax/6)); value/scale rounded to the nearest
    e2m1 magnitude; element 2i in the low nibble of byte i, 2i+1 in the high nibble."""
    N, K = w.shape
    assert K % 32 == 0
    g = w.view(N, K // 32, 32)
    amax = g.abs().amax(dim=2).clamp_min(2.0 ** -100)
    ex = torch.ceil(torch.log2(amax / 6.0)).clamp(-127, 127)
    sb = (ex + 127).to(torch.uint8)
    v = g / torch.exp2(ex).unsqueeze(2)
    mid = torch.tensor(_E2M1_MID, dtype=torch.float32, device=w.device)
    mag = torch.bucketize(v.abs().contiguous(), mid)  # 0..7
    code = (mag.to(torch.uint8) | ((v < 0).to(torch.uint8) << 3)).view(N, K)
    packed = (code[:, 0::2] | (code[:, 1::2] << 4)).contiguous()
    return packed, sb.contiguous()


def _bf16_bits(t: torch.Tensor) -> torch.Tensor:
    return t.to(torch.bfloat16)


def _make_matrix_set(shape: Shape, n: int, N: int, K: int, device, gen) -> tuple:
    """n matrices [N,K] ~ N(0, 0.02^2) in shape.wfmt -> (weights, scales-or-None)."""
    wf = shape.wfmt
    if wf == W_FP32:
        return torch.randn(n, N, K, generator=gen, device=device) * 0.02, None
    if wf == W_BF16:
        out = torch.empty(n, N, K, dtype=torch.bfloat16, device=device)
        for e in range(n):
            out[e] = (torch.randn(N, K, generator=gen, device=device) * 0.02).to(torch.bfloat16)
        return out, None
    if wf == W_FP8E4M3_B128:
        out = torch.empty(n, N, K, dtype=torch.uint8, device=device)
        sc = torch.empty(n, _cdiv(N, 128), _cdiv(K, 128), dtype=torch.float32, device=device)
        for e in range(n):
            out[e], sc[e] = encode_fp8_b128(torch.randn(N, K, generator=gen, device=device) * 0.02)
        return out, sc
    out = torch.empty(n, N, K // 2, dtype=torch.uint8, device=device)
    sc = torch.empty(n, N, K // 32, dtype=torch.uint8, device=device)
    for e in range(n):
        out[e], sc[e] = encode_mxfp4(torch.randn(N, K, generator=gen, device=device) * 0.02)
    return out, sc


def make_expert_weights(shape: Shape, layer: int = 0, device="cpu", seed_tag="w") -> dict:
    """Expert (and shared-expert) weight tensors of one layer, keyed like the C structs."""
    H, I, E = shape.H, shape.I, shape.E
    d = {}
    for name, N, K in (("gate", I, H), ("up", I, H), ("down", H, I)):
        g = _gen(device, shape.name, layer, seed_tag, name)
        d["w_" + name], d["s_" + name] = _make_matrix_set(shape, E, N, K, device, g)
        if shape.n_shared:
            g = _gen(device, shape.name, layer, seed_tag, "sh_" + name)
            d["sh_" + name], d["sh_s_" + name] = _make_matrix_set(shape, shape.n_shared, N, K,
                                                                  device, g)
        else:
            d["sh_" + name], d["sh_s_" + name] = None, None
    return d


# ------------------------------------------------------------ routing inputs

def _act(t: torch.Tensor, shape: Shape) -> torch.Tensor:
    return t.to(torch.bfloat16) if shape.afmt == ACT_BF16 else t.to(torch.float32)


def make_iid_routing(shape: Shape, gamma: int, layer: int = 0, device="cpu", seed_tag="iid"):
    """Dense random router: Wr ~ N(0,0.02^2) (rounded to bf16-representable fp32 unless the
    activations are fp32), x ~ N(0,1).  Returns (router_w [E,H] fp32, x [gamma,H])."""
    g = _gen(device, shape.name, layer, seed_tag, "router")
    wr = torch.randn(shape.E, shape.H, generator=g, device=device) * 0.02
    if shape.afmt == ACT_BF16:
        wr = wr.to(torch.bfloat16).to(torch.float32)
    g = _gen(device, shape.name, layer, seed_tag, "x", gamma)
    x = torch.randn(gamma, shape.H, generator=g, device=device)
    return wr.contiguous(), _act(x, shape).contiguous()


def _carrier(shape: Shape, logits: torch.Tensor, device, gen):
    """Logit carrier: Wr = one-hot rows (Wr[e,e] = 1), x[t,:E] = logits, x[t,E:] ~ N(0,1),
    so the router's logits equal ``logits`` exactly in any precision."""
    gamma = logits.shape[0]
    assert shape.E <= shape.H
    wr = torch.zeros(shape.E, shape.H, dtype=torch.float32, device=device)
    wr[torch.arange(shape.E), torch.arange(shape.E)] = 1.0
    x = torch.randn(gamma, shape.H, generator=gen, device=device)
    x[:, :shape.E] = logits.to(device)
    return wr, _act(x, shape).contiguous()


def make_scattered_routing(shape: Shape, gamma: int, layer: int = 0, device="cpu",
                           seed_tag="scattered"):
    """Every token's E logits iid N(0,1), bf16-rounded, through the logit carrier."""
    g = _gen("cpu", shape.name, layer, seed_tag, "logits", gamma)
    logits = torch.randn(gamma, shape.E, generator=g).to(torch.bfloat16).to(torch.float32)
    gx = _gen(device, shape.name, layer, seed_tag, "x", gamma)
    return _carrier(shape, logits, device, gx)


def make_clustered_routing(shape: Shape, gamma: int, p_copy: float = 0.7, layer: int = 0,
                           device="cpu", seed_tag="clustered"):
    """Draft-tree locality: token t>0 copies the logits of its parent floor((t-1)/2) with
    probability ``p_copy`` (binary tree, token 0 = root), else draws fresh iid logits."""
    g = _gen("cpu", shape.name, layer, seed_tag, "logits", gamma)
    logits = torch.randn(gamma, shape.E, generator=g).to(torch.bfloat16).to(torch.float32)
    coin = torch.rand(gamma, generator=g)
    for t in range(1, gamma):
        if coin[t] < p_copy:
            logits[t] = logits[(t - 1) // 2]
    gx = _gen(device, shape.name, layer, seed_tag, "x", gamma)
    return _carrier(shape, logits, device, gx)


def make_zipf_routing(shape: Shape, gamma: int, alpha: float = 1.0, layer: int = 0, device="cpu",
                      seed_tag="zipf"):
    """Skewed routing (a few hot experts, as in batched verification of similar requests): expert
    of popularity rank r (ranks assigned by a seeded permutation) gets the logit offset
    -alpha * ln(1 + r) on top of iid N(0,1) noise; bf16-rounded, through the logit carrier."""
    g = _gen("cpu", shape.name, layer, seed_tag, "logits", gamma)
    noise = torch.randn(gamma, shape.E, generator=g)
    rs = np.random.RandomState(stream_seed(shape.name, layer, seed_tag, "rank") % (2 ** 31))
    rank = torch.from_numpy(rs.permutation(shape.E).astype(np.float32))
    logits = (noise - alpha * torch.log1p(rank)[None, :]).to(torch.bfloat16).to(torch.float32)
    gx = _gen(device, shape.name, layer, seed_tag, "x", gamma)
    return _carrier(shape, logits, device, gx)


def union_feasible(shape: Shape, gamma: int, U: int) -> bool:
    return shape.top_k <= U <= min(shape.E, gamma * shape.top_k)


def make_exact_union_routing(shape: Shape, gamma: int, U: int, layer: int = 0, device="cpu",
                             seed_tag="exactU"):
    """Logits built so that the expert union has exactly U members.

    The first ceil(U/k) tokens tile [0,U) (coverage); later tokens take seeded random
    k-subsets of [0,U); the j-th chosen expert gets logit 4 - 0.25 j, all others -4;
    finally expert ids go through a seeded permutation so active experts are scattered."""
    k, E = shape.top_k, shape.E
    if not union_feasible(shape, gamma, U):
        raise ValueError(f"union size {U} infeasible for gamma={gamma}, k={k}, E={E}")
    rs = np.random.RandomState(stream_seed(shape.name, layer, seed_tag, gamma, U) % (2 ** 31))
    relabel = rs.permutation(E)
    logits = np.full((gamma, E), -4.0, dtype=np.float32)
    n_tile = _cdiv(U, k)
    for t in range(gamma):
        if t < n_tile:
            chosen = [(t * k + j) % U for j in range(k)]
        else:
            chosen = list(rs.choice(U, size=k, replace=False))
        for j, c in enumerate(chosen):
            logits[t, relabel[c]] = 4.0 - 0.25 * j
    gx = _gen(device, shape.name, layer, seed_tag, "x", gamma, U)
    return _carrier(shape, torch.from_numpy(logits), device, gx)


# ----------------------------------------------------------- host conversion

def to_numpy(t):
    """Raw-storage numpy view of a tensor on the host (bf16 -> uint16)."""
    if t is None:
        return None
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def layer_to_numpy(router_w: torch.Tensor, weights: dict) -> dict:
    d = {"router_w": to_numpy(router_w)}
    for kname, v in weights.items():
        d[kname] = to_numpy(v)
    return d


# ----------------------------------------------------------- draft trees (selection stage)

def make_draft_tree(n_layers: int, E: int, K: int, depth: int = 3, branch: int = 2, seed_tag="tree",
                    p_reuse: float = 0.7):
    """A draft tree like the paper's setup (``depth`` drafting steps, top-``branch`` children
    per node, root = the bonus token) with cumulative draft probabilities and predicted expert
    sets (K experts per layer per node).  A child keeps each of its parent's predicted experts
    with probability ``p_reuse`` (expert locality along a path) and redraws the rest.
    Returns (parent int32 [n], P float32 [n], pred uint32 [n, ceil(n_layers*E/32)])."""
    rs = np.random.RandomState(stream_seed(seed_tag, n_layers, E, K, depth, branch) % (2 ** 31))
    parent, P, sets = [-1], [1.0], []
    sets.append([rs.choice(E, K, replace=False) for _ in range(n_layers)])
    frontier = [0]
    for _ in range(depth):
        nxt = []
        for node in frontier:
            probs = np.sort(rs.dirichlet(np.ones(branch + 1)))[::-1][:branch]
            for b in range(branch):
                parent.append(node)
                P.append(P[node] * float(probs[b]))
                child = []
                for l in range(n_layers):
                    keep = [e for e in sets[node][l] if rs.rand() < p_reuse]
                    pool = [e for e in range(E) if e not in keep]
                    extra = rs.choice(pool, K - len(keep), replace=False) if len(keep) < K else []
                    child.append(np.array(list(keep) + list(extra), dtype=np.int64))
                sets.append(child)
                nxt.append(len(parent) - 1)
        frontier = nxt
    n = len(parent)
    W = _cdiv(n_layers * E, 32)
    pred = np.zeros((n, W), dtype=np.uint32)
    for i in range(n):
        for l in range(n_layers):
            for e in sets[i][l]:
                bit = l * E + int(e)
                pred[i, bit >> 5] |= np.uint32(1 << (bit & 31))
    return np.array(parent, dtype=np.int32), np.array(P, dtype=np.float32), pred


def make_tree_verify_inputs(shape: Shape, parent: np.ndarray, pred: np.ndarray, device="cpu",
                            seed_tag="treex"):
    """Hidden states for the nodes of a draft tree whose single-layer expert sets are given as
    bitmaps (``pred`` uint32 [n, ceil(E/32)], exactly top_k bits per node): through the logit
    carrier, node i routes to exactly the experts of its bitmap (logits 4 - 0.25 j for its j-th
    expert in ascending id, -4 elsewhere).  Returns (router_w [E,H], x [n,H])."""
    n, E, k = len(parent), shape.E, shape.top_k
    logits = np.full((n, E), -4.0, dtype=np.float32)
    for i in range(n):
        ids = [e for e in range(E) if (int(pred[i, e >> 5]) >> (e & 31)) & 1]
        assert len(ids) == k, "one top-k set per node"
        for j, e in enumerate(ids):
            logits[i, e] = 4.0 - 0.25 * j
    gx = _gen(device, shape.name, seed_tag, "x", n)
    return _carrier(shape, torch.from_numpy(logits), device, gx)

"""Seeded synthetic inputs for the METok hot path.

This module only *builds inputs*: planted-event frame features, a text
embedding, attention Q/K with a planted relevance direction, hash-filled
hidden states and K/V caches, class labels.  It holds none of the method's
arithmetic (no similarity, no score, no selection, no budget): both the CUDA
path and the CPU oracle consume what it returns, bit for bit.

All floating inputs are produced as float32 numpy arrays.  For the bf16
configurations every value is first rounded to the nearest bf16 (ties to
even), so widening to float64 (oracle) and narrowing to bf16 (device) are both
exact and the two sides see identical numbers.

The five named configurations follow the workloads the paper evaluates on
(Implementation Details: 32 / 128 frames, 28-layer 7B LLMs with 28 query
heads, 4 KV heads, head dim 128, hidden 3584).  They stand in for the
benchmark videos the paper uses, which are not available here.
"""

from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Optional, Tuple

import numpy as np

# --------------------------------------------------------------------------- #
# configurations
# --------------------------------------------------------------------------- #


@dataclasses.dataclass(frozen=True)
class Config:
    name: str
    index: int            # seed = 1000 + index
    T: int                # frames
    N: int                # visual tokens per frame
    d: int                # vision feature dim (stage 1)
    dtype: str            # "f32" | "bf16"
    k: int                # events
    sigma: float          # per-frame feature noise
    Lt: int               # text query tokens
    Hq: int
    Hkv: int
    dh: int
    D: int                # LLM hidden size
    L: int                # transformer layers holding K/V
    alpha: float          # key-event ratio
    keep_enc: float       # stage-1 key-token keep ratio
    keep_prefill: float   # r of Eq. 6/7
    keep_kv: float        # KV TOPK keep ratio
    n_stages: int         # pruning layers exercised
    kv_text: int          # non-visual rows at the end of the K/V cache
    events: str           # "equal" | "compose" | "uniform" | "zipf"
    static_frac: float = 0.0
    near_dup: bool = False

    @property
    def Nv(self) -> int:
        return self.T * self.N

    @property
    def seed(self) -> int:
        return 1000 + self.index

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2


CONFIGS: Dict[str, Config] = {
    "tiny": Config("tiny", 0, T=8, N=16, d=64, dtype="f32", k=2, sigma=0.05, Lt=4,
                   Hq=1, Hkv=1, dh=64, D=64, L=1, alpha=0.5, keep_enc=0.5,
                   keep_prefill=0.5, keep_kv=0.5, n_stages=1, kv_text=0, events="equal"),
    "frames32": Config("frames32", 1, T=32, N=144, d=1024, dtype="bf16", k=4, sigma=0.1, Lt=16,
                      Hq=28, Hkv=4, dh=128, D=3584, L=28, alpha=0.5, keep_enc=0.3,
                      keep_prefill=0.5, keep_kv=0.1, n_stages=2, kv_text=16, events="compose"),
    "frames64": Config("frames64", 2, T=64, N=196, d=1152, dtype="bf16", k=8, sigma=0.1, Lt=32,
                      Hq=28, Hkv=4, dh=128, D=3584, L=28, alpha=0.5, keep_enc=0.25,
                      keep_prefill=0.5, keep_kv=0.1, n_stages=3, kv_text=32, events="compose",
                      near_dup=True),
    "frames128": Config("frames128", 3, T=128, N=144, d=3584, dtype="bf16", k=16, sigma=0.1, Lt=64,
                       Hq=28, Hkv=4, dh=128, D=3584, L=28, alpha=0.5, keep_enc=0.2,
                       keep_prefill=0.5, keep_kv=0.065, n_stages=3, kv_text=64, events="uniform"),
    "stress": Config("stress", 4, T=512, N=144, d=1024, dtype="bf16", k=64, sigma=0.1, Lt=128,
                     Hq=28, Hkv=4, dh=128, D=3584, L=28, alpha=0.5, keep_enc=0.2,
                     keep_prefill=0.5, keep_kv=0.1, n_stages=3, kv_text=128, events="zipf",
                     static_frac=0.05),
}
# the 128-frame workload with the vision tower's own feature width
CONFIGS["frames128d1024"] = dataclasses.replace(CONFIGS["frames128"], name="frames128d1024", d=1024)

# The paper's two other model sizes (Implementation Details): 32 frames of 196 tokens into a 24-layer
# decoder with 14 query / 2 key-value heads of 64, k = 5, r = 0.76; and 16 frames of 196 tokens into a
# 40-layer decoder with 40 heads of 128 and no head sharing, k = 3, r = 0.65, L_H = [13, 24, 34].
CONFIGS["small24"] = Config("small24", 5, T=32, N=196, d=1152, dtype="bf16", k=5, sigma=0.1, Lt=24,
                            Hq=14, Hkv=2, dh=64, D=896, L=24, alpha=0.5, keep_enc=0.25,
                            keep_prefill=0.76, keep_kv=0.1, n_stages=3, kv_text=24, events="compose")
CONFIGS["large40"] = Config("large40", 6, T=16, N=196, d=1152, dtype="bf16", k=3, sigma=0.1, Lt=40,
                            Hq=40, Hkv=40, dh=128, D=5120, L=40, alpha=0.5, keep_enc=0.25,
                            keep_prefill=0.65, keep_kv=0.1, n_stages=3, kv_text=40, events="compose")

CONFIG_ORDER = ["tiny", "frames32", "frames64", "frames128", "stress"]


def rng_for(cfg: Config, part: int) -> np.random.Generator:
    """Independent stream per (config, part) so parts can be built in any order."""
    return np.random.default_rng([cfg.seed, part])


# --------------------------------------------------------------------------- #
# number formats
# --------------------------------------------------------------------------- #


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """float32 -> nearest bf16 (ties to even), returned as float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    bias = np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    r = (u + bias) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 holding bf16-representable values -> uint16 bit patterns."""
    return (np.ascontiguousarray(x, dtype=np.float32).view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def quantize(x: np.ndarray, dtype: str) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float32)
    return round_to_bf16(x) if dtype == "bf16" else x


# --------------------------------------------------------------------------- #
# events
# --------------------------------------------------------------------------- #


def _compose(total: int, parts: int, lo: int, rng: np.random.Generator) -> List[int]:
    """Random composition of `total` into `parts` integers, each >= lo."""
    free = total - parts * lo
    assert free >= 0
    cuts = np.sort(rng.integers(0, free + 1, size=parts - 1))
    edges = np.concatenate([[0], cuts, [free]])
    return [int(edges[i + 1] - edges[i]) + lo for i in range(parts)]


def event_lengths(cfg: Config) -> List[int]:
    rng = rng_for(cfg, 1)
    if cfg.events == "equal":
        assert cfg.T % cfg.k == 0
        return [cfg.T // cfg.k] * cfg.k
    if cfg.events == "compose":
        return _compose(cfg.T, cfg.k, 2, rng)
    if cfg.events == "uniform":
        lens = [int(v) for v in rng.integers(2, 17, size=cfg.k)]
        while sum(lens) > cfg.T:
            i = int(np.argmax(lens))
            lens[i] -= 1
        while sum(lens) < cfg.T:
            i = int(np.argmin(lens))
            lens[i] += 1
        assert all(2 <= v <= 16 for v in lens)
        return lens
    if cfg.events == "zipf":
        h = sum(1.0 / i for i in range(1, cfg.k + 1))
        lens = [max(1, int(round(cfg.T * (1.0 / i) / h))) for i in range(1, cfg.k + 1)]
        while sum(lens) > cfg.T:
            i = int(np.argmax(lens))
            lens[i] -= 1
        while sum(lens) < cfg.T:
            lens[0] += 1
        order = rng.permutation(cfg.k)
        return [lens[int(i)] for i in order]
    raise ValueError(cfg.events)


def offsets_from_lengths(lens: List[int]) -> np.ndarray:
    return np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)


# --------------------------------------------------------------------------- #
# stage 1: frame features and text embedding
# --------------------------------------------------------------------------- #


def vision_inputs(cfg: Config) -> Dict[str, object]:
    """Planted-event features V[T,N,d], text embedding t[d], and what was planted."""
    lens = event_lengths(cfg)
    offs = offsets_from_lengths(lens)
    rng_b = rng_for(cfg, 2)
    rng_n = rng_for(cfg, 3)
    rng_t = rng_for(cfg, 4)

    base = rng_b.standard_normal((cfg.k, cfg.N, cfg.d), dtype=np.float32)
    near_dup_at = None
    near_dup_event = None
    if cfg.near_dup:
        # one boundary whose two sides stay 0.98-similar
        e = 1 + int(rng_b.integers(0, cfg.k - 1))
        c = min(0.98 * (1.0 + cfg.sigma ** 2), 0.9999)
        fresh = rng_b.standard_normal((cfg.N, cfg.d), dtype=np.float32)
        base[e] = np.float32(c) * base[e - 1] + np.float32(math.sqrt(1.0 - c * c)) * fresh
        near_dup_at = int(offs[e]) - 1          # split after this frame
        near_dup_event = e
    static_pos = np.zeros(0, dtype=np.int64)
    if cfg.static_frac > 0:
        n_static = max(1, int(round(cfg.static_frac * cfg.N)))
        static_pos = np.sort(rng_b.choice(cfg.N, size=n_static, replace=False))
        shared = rng_b.standard_normal((cfg.d,), dtype=np.float32)
        base[:, static_pos, :] = shared

    # planted relevance: the relevant events carry a common direction w, and the
    # text embedding points along w (10 % relative noise)
    n_rel = int(math.ceil(cfg.alpha * cfg.k - 1e-9))
    if near_dup_event is not None and n_rel >= 2:
        # the two near-duplicate events are equally relevant by construction: plant both
        others = np.array([e for e in range(cfg.k) if e not in (near_dup_event - 1, near_dup_event)])
        pick = rng_t.choice(others, size=n_rel - 2, replace=False)
        relevant = np.sort(np.concatenate([pick, [near_dup_event - 1, near_dup_event]])).astype(np.int32)
    else:
        relevant = np.sort(rng_t.choice(cfg.k, size=n_rel, replace=False)).astype(np.int32)
    w = rng_t.standard_normal(cfg.d)
    w /= np.linalg.norm(w)
    amp = 0.25 * math.sqrt(cfg.d)
    live = np.setdiff1d(np.arange(cfg.N), static_pos)
    for e in relevant:
        base[e, live, :] += (amp * w).astype(np.float32)[None, :]
    t = 3.0 * (w + (0.1 / math.sqrt(cfg.d)) * rng_t.standard_normal(cfg.d))
    t = quantize(t.astype(np.float32), cfg.dtype)

    V = np.empty((cfg.T, cfg.N, cfg.d), dtype=np.float32)
    for e in range(cfg.k):
        f0, f1 = int(offs[e]), int(offs[e + 1])
        noise = rng_n.standard_normal((f1 - f0, cfg.N, cfg.d), dtype=np.float32)
        V[f0:f1] = base[e][None] + np.float32(cfg.sigma) * noise
    V = quantize(V, cfg.dtype)

    return {
        "V": V, "t": t, "lengths": lens, "event_offsets": offs,
        "boundaries": (offs[1:-1] - 1).astype(np.int32),
        "relevant_events": relevant, "near_dup_boundary": near_dup_at,
        "static_positions": static_pos,
    }


def frame_is_relevant(cfg: Config, vis: Dict[str, object]) -> np.ndarray:
    """bool[T]: frame belongs to one of the planted relevant events."""
    offs = vis["event_offsets"]
    out = np.zeros(cfg.T, dtype=bool)
    for e in vis["relevant_events"]:
        out[int(offs[e]):int(offs[e + 1])] = True
    return out


# --------------------------------------------------------------------------- #
# stage 2: prefill Q/K, hidden states, classes
# --------------------------------------------------------------------------- #


def token_groups(cfg: Config, n_vis: int, n_key: Optional[int] = None, stage: int = 1,
                 vis: Optional[Dict[str, object]] = None) -> np.ndarray:
    """int32[n_vis] class of each visual token: 0 = key-event token, 1 = non-key.

    With `vis` given (and n_vis == T*N) the class follows the planted relevant
    events frame by frame; otherwise exactly `n_key` tokens, placed by the seed,
    are class 0.
    """
    if vis is not None and n_vis == cfg.Nv:
        rel = frame_is_relevant(cfg, vis)
        return np.repeat(np.where(rel, 0, 1).astype(np.int32), cfg.N)
    assert n_key is not None and 0 <= n_key <= n_vis
    rng = rng_for(cfg, 20 + stage)
    g = np.ones(n_vis, dtype=np.int32)
    g[rng.permutation(n_vis)[:n_key]] = 0
    return g


def prefill_inputs(cfg: Config, stage: int, n_vis: int, groups: np.ndarray, vis_start: int = 0,
                   planted: bool = True) -> Dict[str, object]:
    """Q_text[Hq,Lt,dh], K[Hkv,S,dh] for one pruning layer; S = vis_start + n_vis + Lt."""
    rng = rng_for(cfg, 30 + stage)
    S = vis_start + n_vis + cfg.Lt
    sd = np.float32(cfg.dh ** -0.5)
    if cfg.name == "tiny":
        sd = np.float32(1.0)
    Q = sd * rng.standard_normal((cfg.Hq, cfg.Lt, cfg.dh), dtype=np.float32)
    K = sd * rng.standard_normal((cfg.Hkv, S, cfg.dh), dtype=np.float32)
    if planted:
        c = math.sqrt(2.0 * math.sqrt(cfg.dh))
        rho = 0.5 * np.where(groups == 0, 1.0, -1.0) + rng.standard_normal(n_vis)
        rep = cfg.Hq // cfg.Hkv
        for g in range(cfg.Hkv):
            u = rng.standard_normal(cfg.dh)
            u /= np.linalg.norm(u)
            K[g, vis_start:vis_start + n_vis, :] += (c * rho[:, None] * u[None, :]).astype(np.float32)
            Q[g * rep:(g + 1) * rep] += (c * u).astype(np.float32)[None, None, :]
    return {"Q": quantize(Q, cfg.dtype), "K": quantize(K, cfg.dtype), "S": S,
            "vis_start": vis_start, "n_vis": n_vis}


# --------------------------------------------------------------------------- #
# hash-filled payloads (hidden states, K/V caches): content only has to be
# position-distinct, and must be reproducible row by row without holding the
# whole tensor on the host.
# --------------------------------------------------------------------------- #


def _mix_np(idx: np.ndarray, salt: int) -> np.ndarray:
    m = np.uint64(0xFFFFFFFF)
    h = (idx.astype(np.uint64) & m) * np.uint64(0x1E3779B1) + np.uint64((salt * 0x05EBCA77 + 0x1234567) & 0xFFFFFFFF)
    h &= m
    h ^= h >> np.uint64(15)
    h = (h * np.uint64(0x2C1B3C6D)) & m
    h ^= h >> np.uint64(12)
    return h


def payload_rows_np(salt: int, rows: np.ndarray, width: int, dtype: str) -> np.ndarray:
    """Rows `rows` of the hash-filled [*, width] payload with this salt.

    bf16: uint16 bit patterns (top exponent bit cleared: finite, |x| < 2);
    f32: float32 values j/64 with j in [0, 4096).
    """
    rows = np.asarray(rows, dtype=np.int64)
    idx = rows[:, None] * width + np.arange(width, dtype=np.int64)[None, :]
    h = _mix_np(idx, salt)
    if dtype == "bf16":
        return (h & np.uint64(0xBFFF)).astype(np.uint16)
    return ((h & np.uint64(0xFFF)).astype(np.float32) / np.float32(64.0)).astype(np.float32)


def payload_torch(salt: int, n_rows: int, width: int, dtype: str, device):
    """The same payload as a torch tensor on `device` (bf16 or float32)."""
    import torch

    out = torch.empty((n_rows, width), dtype=torch.bfloat16 if dtype == "bf16" else torch.float32,
                      device=device)
    step = max(1, (1 << 24) // width)
    add = (salt * 0x05EBCA77 + 0x1234567) & 0xFFFFFFFF
    for r0 in range(0, n_rows, step):
        r1 = min(n_rows, r0 + step)
        idx = torch.arange(r0 * width, r1 * width, dtype=torch.int64, device=device)
        h = ((idx & 0xFFFFFFFF) * 0x1E3779B1 + add) & 0xFFFFFFFF
        h ^= h >> 15
        h = (h * 0x2C1B3C6D) & 0xFFFFFFFF
        h ^= h >> 12
        if dtype == "bf16":
            bits = (h & 0xBFFF).to(torch.int32)
            bits = torch.where(bits >= 32768, bits - 65536, bits).to(torch.int16)
            out[r0:r1] = bits.view(torch.bfloat16).view(r1 - r0, width)
        else:
            out[r0:r1] = ((h & 0xFFF).to(torch.float32) / 64.0).view(r1 - r0, width)
    return out


def hidden_salt(cfg: Config, stage: int) -> int:
    return 7000 + 16 * cfg.index + stage


def kv_salt(cfg: Config, layer: int, which: int, head: int) -> int:
    """which: 0 = K, 1 = V."""
    return 100000 * (cfg.index + 1) + (layer * 2 + which) * cfg.Hkv + head


def kv_cache_torch(cfg: Config, device, layers: Optional[int] = None):
    """Per-layer K and V caches [Hkv, S_cap, dh], S_cap = Nv + kv_text."""
    import torch

    L = cfg.L if layers is None else layers
    S_cap = cfg.Nv + cfg.kv_text
    ks, vs = [], []
    for layer in range(L):
        for which, dst in ((0, ks), (1, vs)):
            slabs = [payload_torch(kv_salt(cfg, layer, which, h), S_cap, cfg.dh, cfg.dtype, device)
                     for h in range(cfg.Hkv)]
            dst.append(torch.stack(slabs, dim=0).contiguous())
    return ks, vs


def kv_scores(cfg: Config, n_vis: int, per_layer: bool = False, layers: Optional[int] = None) -> np.ndarray:
    """Positive, tie-free visual-token scores for the KV TOPK policy (float32)."""
    rng = rng_for(cfg, 50)
    L = (cfg.L if layers is None else layers) if per_layer else 1
    s = np.exp(rng.standard_normal((L, n_vis))).astype(np.float32) / np.float32(n_vis)
    return s if per_layer else s[0]

"""CPU oracle for the METok hot path.  TEST INFRASTRUCTURE ONLY.

A plain, slow restatement in float64 numpy of what each step of the path
computes, written from the paper's definitions (Eq. 4, 5, 6, 7, Algorithm 1,
the KV rule of the "Decoding" subsection) and, where the paper is silent, from
the readings listed at the top of each function.  Nothing here is tuned, tiled,
fused or reordered.  It shares no code with the CUDA library and imports
nothing from it; only tests, the smoke check and the benchmark's CPU-baseline
leg may call it.  The product path never does.

Conventions
  * inputs arrive as numpy arrays of any float type and are widened to float64
    exactly; index outputs are int32/int64 numpy arrays;
  * every ordering is a stable full sort with "lower index wins" on ties, so
    each result is unique;
  * counts derived from a ratio use ``ceilq(x) = ceil(x - 1e-9)`` with the ratio
    and the product held in float64 (the C ABI carries ratios as double, so a
    printed ratio such as r = 0.55 of 1000 tokens gives 550, not 551);
  * every norm is clamped below by EPS = 1e-8.

Pins: every function below is pinned in tests/test_oracle_*.py against planted
structure, closed forms, brute force on tiny inputs, independent float64
restatements with library routines, constants printed in the paper, and
invariants; none is left unpinned.  The oracle's answers are unique (exact
float64 arithmetic on the inputs, lower index on exact ties).  What the GPU
comparison tolerates is a separate matter: where the deciding gap of an index
decision is below 1e-3 relative (a score against its top-k threshold, the best
against the second-best cosine of a merge assignment) the kernel's bf16 / fp32
rounding may decide the other way; ``near_threshold`` and the ``margin`` of
``merge_assign`` report those cases (both pinned by construction), and the
parity tests count them against ceilings.
"""

from __future__ import annotations

import math
from typing import Dict, List, Optional, Sequence

import numpy as np

EPS = 1e-8
NEAR_TIE = 1e-3

SIM_FLATTEN = 0
SIM_MEANPOOL = 1
AGG_MEAN = 0
AGG_MAX = 1
KV_PAPER = 0
KV_TOPK = 1
KV_GIVEN = 2


# --------------------------------------------------------------------------- #
# small shared definitions
# --------------------------------------------------------------------------- #


def f32(x: float) -> float:
    """The softmax scale as the C ABI carries it: float32, widened."""
    return float(np.float32(x))


def ceilq(x: float) -> int:
    """Ceiling used for every count derived from a ratio (the paper shows only
    the ceiling form, for the key-event count)."""
    return int(math.ceil(x - 1e-9))


def round_bf16(x: np.ndarray) -> np.ndarray:
    """float64 -> nearest value with an 8-bit significand (bf16), ties to even.
    Normal range only, which is all the features ever reach."""
    x = np.asarray(x, dtype=np.float64)
    m, e = np.frexp(x)                       # x = m * 2**e, 0.5 <= |m| < 1
    return np.ldexp(np.rint(m * 256.0), e - 8)


def round_out(x: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == "bf16":
        return round_bf16(x)
    return np.asarray(x, dtype=np.float64).astype(np.float32).astype(np.float64)


def near_threshold(s: np.ndarray, tau: float) -> np.ndarray:
    """Near-tie band of a top-k decision: scores within 1e-3 (relative to the
    threshold score tau, the last one kept) of the threshold.  For thresholds
    close to zero the band is floored at 1e-3 of 1e-3 of the largest |score|."""
    floor = NEAR_TIE * max(float(np.max(np.abs(s))), 1e-300)
    return np.abs(s - tau) < NEAR_TIE * max(abs(float(tau)), floor)


def _order_desc(score: np.ndarray) -> np.ndarray:
    """Indices sorted by (score descending, index ascending)."""
    return np.lexsort((np.arange(score.size), -score))


def _order_asc(score: np.ndarray) -> np.ndarray:
    return np.lexsort((np.arange(score.size), score))


# --------------------------------------------------------------------------- #
# a1: temporal event segmentation (Eq. 4; Algorithm 1, "Event temporal segmentation")
# --------------------------------------------------------------------------- #


def frame_similarity(V: np.ndarray, sim_mode: int = SIM_FLATTEN) -> np.ndarray:
    """S_i = cos(v_i, v_{i+1}) for i = 0..T-2 (Eq. 4).

    Readings: there are T-1 adjacent pairs (the equation's index range names T).
    v_i is an N x d matrix; FLATTEN takes the Frobenius inner product over all
    N*d entries and Frobenius norms; MEANPOOL first averages the N tokens.
    """
    V = np.asarray(V, dtype=np.float64)
    T = V.shape[0]
    a = V.reshape(T, -1) if sim_mode == SIM_FLATTEN else V.mean(axis=1)
    norms = np.maximum(np.sqrt(np.sum(a * a, axis=1)), EPS)
    sims = np.empty(max(T - 1, 0), dtype=np.float64)
    for i in range(T - 1):
        sims[i] = np.sum(a[i] * a[i + 1]) / (norms[i] * norms[i + 1])
    return sims


def split_events(sims: np.ndarray, k: int) -> Dict[str, np.ndarray]:
    """Boundaries = the k-1 lowest S_i (lower i wins ties); events = the runs
    between them.  No minimum event length."""
    T = sims.size + 1
    assert 1 <= k <= T
    lowest = _order_asc(sims)[: k - 1]
    boundaries = np.sort(lowest).astype(np.int32)        # split between frame b and b+1
    offsets = np.concatenate([[0], boundaries + 1, [T]]).astype(np.int32)
    frame_event = np.zeros(T, dtype=np.int32)
    for e in range(k):
        frame_event[offsets[e]:offsets[e + 1]] = e
    return {"boundaries": boundaries, "event_offsets": offsets, "frame_event": frame_event}


def segment_events(V: np.ndarray, k: int, sim_mode: int = SIM_FLATTEN) -> Dict[str, np.ndarray]:
    sims = frame_similarity(V, sim_mode)
    out = split_events(sims, k)
    out["sims"] = sims
    return out


# --------------------------------------------------------------------------- #
# a2: text relevance and key events (Eq. 5; Algorithm 1, "Key semantic identification")
# --------------------------------------------------------------------------- #


def token_relevance(V: np.ndarray, t: np.ndarray) -> np.ndarray:
    """s_j = cos(x_j, t) per visual token (Eq. 5 read per token: v_i t^T has one
    entry per token, each divided by that token's norm and by ||t||)."""
    X = np.asarray(V, dtype=np.float64).reshape(-1, V.shape[-1])
    t = np.asarray(t, dtype=np.float64).reshape(-1)
    tn = max(math.sqrt(float(np.sum(t * t))), EPS)
    xn = np.maximum(np.sqrt(np.sum(X * X, axis=1)), EPS)
    return (X @ t) / (xn * tn)


def key_events(token_score: np.ndarray, T: int, N: int, event_offsets: np.ndarray, alpha: float,
               event_agg: int = AGG_MEAN) -> Dict[str, np.ndarray]:
    """Frame score = mean of its N token scores; event score = mean over the
    event's frames (body text) or max (Algorithm 1); key events = the
    ceil(alpha*k) best, lower event index winning ties."""
    k = len(event_offsets) - 1
    frame_score = token_score.reshape(T, N).mean(axis=1)
    event_score = np.empty(k, dtype=np.float64)
    for e in range(k):
        fs = frame_score[event_offsets[e]:event_offsets[e + 1]]
        event_score[e] = fs.mean() if event_agg == AGG_MEAN else fs.max()
    n_key = min(k, ceilq(float(alpha) * k))
    is_key = np.zeros(k, dtype=np.uint8)
    is_key[_order_desc(event_score)[:n_key]] = 1
    return {"frame_score": frame_score, "event_score": event_score, "event_is_key": is_key}


# --------------------------------------------------------------------------- #
# a3: per-event key-token top-k  (the paper is silent; defined from Eq. 5's
# relevance, the event partition, and the ceiling convention)
# --------------------------------------------------------------------------- #


def event_token_budget(m_e: int, ratio: float) -> int:
    return min(m_e, max(1, ceilq(float(ratio) * m_e)))


def key_token_topk(token_score: np.ndarray, N: int, event_offsets: np.ndarray, event_is_key: np.ndarray,
                   keep_key: float, keep_nonkey: float) -> Dict[str, np.ndarray]:
    """In event e keep the k_e highest-scored tokens (ties: lower token index)."""
    k = len(event_offsets) - 1
    Nv = token_score.size
    is_key_token = np.zeros(Nv, dtype=np.uint8)
    near = np.zeros(Nv, dtype=bool)
    budgets = np.zeros(k, dtype=np.int32)
    for e in range(k):
        lo, hi = int(event_offsets[e]) * N, int(event_offsets[e + 1]) * N
        s = token_score[lo:hi]
        k_e = event_token_budget(hi - lo, keep_key if event_is_key[e] else keep_nonkey)
        budgets[e] = k_e
        order = _order_desc(s)
        is_key_token[lo + order[:k_e]] = 1
        near[lo:hi] = near_threshold(s, s[order[k_e - 1]])
    key_idx = np.nonzero(is_key_token)[0].astype(np.int32)
    return {"is_key_token": is_key_token, "key_idx": key_idx, "event_budget": budgets, "near_tie": near}


# --------------------------------------------------------------------------- #
# a4: merge-assign and averaging (the paper is silent; see a3)
# --------------------------------------------------------------------------- #


def merge_assign(V: np.ndarray, N: int, event_offsets: np.ndarray, is_key_token: np.ndarray,
                 dtype: str) -> Dict[str, np.ndarray]:
    """Every non-key token joins the key token of its own event with the highest
    cosine similarity (ties: lower key index).  Output token c = plain mean of
    key token c and its members, in original feature space, rounded once."""
    X = np.asarray(V, dtype=np.float64).reshape(-1, V.shape[-1])
    Nv, d = X.shape
    k = len(event_offsets) - 1
    key_idx = np.nonzero(is_key_token)[0]
    n_out = key_idx.size
    slot_of = -np.ones(Nv, dtype=np.int64)
    slot_of[key_idx] = np.arange(n_out)
    assign = np.empty(Nv, dtype=np.int32)
    margin = np.full(Nv, np.inf)
    out_event = np.empty(n_out, dtype=np.int32)
    norms = np.maximum(np.sqrt(np.sum(X * X, axis=1)), EPS)
    for e in range(k):
        lo, hi = int(event_offsets[e]) * N, int(event_offsets[e + 1]) * N
        idx = np.arange(lo, hi)
        keys = idx[is_key_token[lo:hi] == 1]
        rest = idx[is_key_token[lo:hi] == 0]
        out_event[slot_of[keys]] = e
        assign[keys] = slot_of[keys]
        if rest.size == 0:
            continue
        cos = (X[rest] @ X[keys].T) / (norms[rest][:, None] * norms[keys][None, :])
        best = np.argmax(cos, axis=1)                  # first maximum = lower key index
        assign[rest] = slot_of[keys[best]]
        if keys.size > 1:
            top2 = np.partition(cos, keys.size - 2, axis=1)[:, -2:]
            b, s2 = top2[:, 1], top2[:, 0]
            margin[rest] = (b - s2) / np.maximum(np.abs(b), 1e-300)
    members = np.bincount(assign, minlength=n_out).astype(np.int32)
    sums = np.zeros((n_out, d), dtype=np.float64)
    for j in range(Nv):
        sums[assign[j]] += X[j]
    mean = sums / members[:, None]
    return {"out_feats_exact": mean, "out_feats": round_out(mean, dtype),
            "out_src": key_idx.astype(np.int32), "out_event": out_event, "out_members": members,
            "assign": assign, "margin": margin, "n_out": n_out}


def compress_vision(V: np.ndarray, t: np.ndarray, event_offsets: np.ndarray, alpha: float,
                    keep_key: float, keep_nonkey: float, dtype: str,
                    event_agg: int = AGG_MEAN, key_events_given: Optional[np.ndarray] = None) -> Dict[str, np.ndarray]:
    """a2 + a3 + a4 chained, as the library's stage-1 call runs them.  `key_events_given` (bool [k])
    replaces Eq. 5's choice of key events: the ablation with randomly chosen key events."""
    T, N, _ = V.shape
    s = token_relevance(V, t)
    ev = key_events(s, T, N, event_offsets, alpha, event_agg)
    if key_events_given is not None:
        ev["event_is_key"] = np.asarray(key_events_given).astype(ev["event_is_key"].dtype)
    sel = key_token_topk(s, N, event_offsets, ev["event_is_key"], keep_key, keep_nonkey)
    mer = merge_assign(V, N, event_offsets, sel["is_key_token"], dtype)
    out = {"token_score": s}
    out.update(ev)
    out.update(sel)
    out.update(mer)
    return out


# --------------------------------------------------------------------------- #
# NEXT: the paper's own stage-1 compressor -- key frames and adaptive pooling
# (Algorithm 1, "Adaptive pooling strategy")
# --------------------------------------------------------------------------- #


def key_frames(frame_score: np.ndarray, event_offsets: np.ndarray, beta: float) -> np.ndarray:
    """Per event the ceil(beta*|E_j|) best-scored frames are key frames."""
    T = frame_score.size
    is_key = np.zeros(T, dtype=np.uint8)
    for e in range(len(event_offsets) - 1):
        lo, hi = int(event_offsets[e]), int(event_offsets[e + 1])
        n = min(hi - lo, max(1, ceilq(float(beta) * (hi - lo))))
        is_key[lo + _order_desc(frame_score[lo:hi])[:n]] = 1
    return is_key


def pool2d(frame: np.ndarray, G: int, s: int) -> np.ndarray:
    """Average pooling of a G x G token grid, window = stride = s, output side
    ceil(G/s); edge windows average only the cells that exist."""
    d = frame.shape[-1]
    g = np.asarray(frame, dtype=np.float64).reshape(G, G, d)
    Go = -(-G // s)
    out = np.empty((Go, Go, d), dtype=np.float64)
    for a in range(Go):
        for b in range(Go):
            win = g[a * s:min(G, (a + 1) * s), b * s:min(G, (b + 1) * s)]
            out[a, b] = win.reshape(-1, d).mean(axis=0)
    return out.reshape(Go * Go, d)


def adaptive_pool(V: np.ndarray, t: np.ndarray, event_offsets: np.ndarray, alpha: float, beta: float,
                  strides: Sequence[int], dtype: str, event_agg: int = AGG_MEAN,
                  key_frames_given: Optional[np.ndarray] = None) -> Dict[str, np.ndarray]:
    """strides = (s1, s2, s1_nonkey, s2_nonkey): key/non-key frames of key events,
    then of non-key events.  Frames are pooled and appended in temporal order.
    `key_frames_given` (bool [T]) replaces the scored choice of key frames: the ablation
    with randomly chosen key frames."""
    T, N, d = V.shape
    G = int(round(math.sqrt(N)))
    assert G * G == N
    s = token_relevance(V, t)
    ev = key_events(s, T, N, event_offsets, alpha, event_agg)
    kf = key_frames(ev["frame_score"], event_offsets, beta)
    if key_frames_given is not None:
        kf = np.asarray(key_frames_given).astype(kf.dtype)
    frame_stride = np.empty(T, dtype=np.int32)
    for e in range(len(event_offsets) - 1):
        for f in range(int(event_offsets[e]), int(event_offsets[e + 1])):
            if ev["event_is_key"][e]:
                frame_stride[f] = strides[0] if kf[f] else strides[1]
            else:
                frame_stride[f] = strides[2] if kf[f] else strides[3]
    chunks, out_frame = [], []
    for f in range(T):
        p = pool2d(V[f], G, int(frame_stride[f]))
        chunks.append(p)
        out_frame.append(np.full(p.shape[0], f, dtype=np.int32))
    feats = np.concatenate(chunks, axis=0)
    out = {"token_score": s, "frame_is_key": kf, "frame_stride": frame_stride,
           "out_feats_exact": feats, "out_feats": round_out(feats, dtype),
           "out_frame": np.concatenate(out_frame), "n_out": feats.shape[0]}
    out.update(ev)
    return out


# --------------------------------------------------------------------------- #
# a5: text -> visual attention score at a pruning layer
# ("Hierarchical Token Pruning"; attention form and scale of Eq. 2)
# --------------------------------------------------------------------------- #


def attention_scores(Q: np.ndarray, K: np.ndarray, vis_start: int, n_vis: int,
                     softmax_scale: float) -> np.ndarray:
    """a_j = mean over all heads h and text queries q of softmax_u(Q[h,q].K[g(h),u] * scale)[j].

    Readings: post-softmax probabilities; the Lt text queries occupy the last Lt
    positions; query q sees keys u <= S - Lt + q (causal), which covers every
    visual token; heads share KV heads in contiguous groups, g(h) = h // (Hq/Hkv).
    """
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    Hq, Lt, dh = Q.shape
    Hkv, S, _ = K.shape
    rep = Hq // Hkv
    scale = f32(softmax_scale)
    text_start = S - Lt
    acc = np.zeros(n_vis, dtype=np.float64)
    u = np.arange(S)[None, :]
    visible = u <= (text_start + np.arange(Lt))[:, None]   # [Lt, S]
    for h in range(Hq):
        g = h // rep
        logits = (Q[h] @ K[g].T) * scale                  # [Lt, S]
        logits = np.where(visible, logits, -np.inf)
        p = np.exp(logits - logits.max(axis=1, keepdims=True))
        p /= p.sum(axis=1, keepdims=True)
        acc += p[:, vis_start:vis_start + n_vis].sum(axis=0)
    return acc / (Hq * Lt)


# --------------------------------------------------------------------------- #
# a6: retention schedule (Eq. 6, 7) and event-weighted top-k
# --------------------------------------------------------------------------- #


def retention_ratios(alpha: float, r: float, stage: int):
    """(R_key, R_non-key) after pruning layer l_stage.  Eq. 6 leaves l = l3 and
    Eq. 7 leaves l = l2 unassigned; both are read as the next case (0)."""
    a, r = float(alpha), float(r)
    if stage == 0:
        return 1.0, 1.0
    if stage == 1:
        return r, a * r
    if stage == 2:
        return r * r, 0.0
    if stage == 3:
        return 0.0, 0.0
    raise ValueError(stage)


def retention_budgets(alpha: float, r: float, stage: int, N0: Sequence[int]) -> np.ndarray:
    """Token budgets relative to the counts N0 = (key, non-key) first passed
    into the LLM."""
    rk, rn = retention_ratios(alpha, r, stage)
    return np.array([min(N0[0], ceilq(rk * N0[0])), min(N0[1], ceilq(rn * N0[1]))], dtype=np.int32)


def weighted_topk(scores: np.ndarray, token_group: np.ndarray, group_budget: Sequence[int], S: int,
                  vis_start: int) -> Dict[str, np.ndarray]:
    """Keep, in each class g, the min(population, budget_g) best-scored visual
    tokens (ties: lower index); keep every non-visual position; ascending."""
    scores = np.asarray(scores, dtype=np.float64)
    n_vis = scores.size
    keep_vis = np.zeros(n_vis, dtype=bool)
    near = np.zeros(n_vis, dtype=bool)
    for g, budget in enumerate(group_budget):
        idx = np.nonzero(token_group == g)[0]
        n = min(idx.size, int(budget))
        if n <= 0 or idx.size == 0:
            continue
        s = scores[idx]
        order = _order_desc(s)
        keep_vis[idx[order[:n]]] = True
        if n < idx.size:
            near[idx] = near_threshold(s, s[order[n - 1]])
    keep = np.ones(S, dtype=bool)
    keep[vis_start:vis_start + n_vis] = keep_vis
    keep_idx = np.nonzero(keep)[0].astype(np.int32)
    return {"keep_idx": keep_idx, "S_out": keep_idx.size, "near_tie": near}


def prune_schedule(Qs: Sequence[np.ndarray], Ks: Sequence[np.ndarray], token_group: np.ndarray, alpha: float,
                   r: float, vis_start: int, softmax_scale: float) -> List[Dict[str, np.ndarray]]:
    """The pruning levels l1, l2, l3 one after the other (section 3.2.2): level s scores the visual
    tokens that survived level s-1 with that layer's text queries and keys (Qs[s], Ks[s]: rows of
    the survivors, in order), and keeps per class the budget of Eq. 6/7 for stage s, which is
    relative to the class counts N0 at the first level.  A survivor keeps its class.  Per level:
    the level's result plus `token_group` (its input classes) and `origin` (for each of its visual
    tokens the index among the first level's)."""
    group = np.asarray(token_group, dtype=np.int32)
    N0 = [int((group == 0).sum()), int((group == 1).sum())]
    origin = np.arange(group.size, dtype=np.int32)
    levels = []
    for s, (Q, K) in enumerate(zip(Qs, Ks), start=1):
        n_vis = group.size
        S = K.shape[1]
        a = attention_scores(Q, K, vis_start, n_vis, softmax_scale)
        budget = retention_budgets(alpha, r, s, N0)
        sel = weighted_topk(a, group, budget, S, vis_start)
        sel.update({"scores": a, "token_group": group, "origin": origin, "budget": budget})
        levels.append(sel)
        kept_vis = sel["keep_idx"][(sel["keep_idx"] >= vis_start) & (sel["keep_idx"] < vis_start + n_vis)] - vis_start
        group, origin = group[kept_vis], origin[kept_vis]
    return levels


def schedule_kv_lists(levels: List[Dict[str, np.ndarray]], level_layer: Sequence[int], L: int,
                      S: int) -> List[np.ndarray]:
    """K/V keep lists in line with the hierarchical pruning (section 3.3): layer l lies in group
    g = #{s : level_layer[s] <= l}; its cache holds the rows of level g's input and keeps what level
    g + 1 kept; layers at or beyond the last pruning layer keep all their rows.  `levels` is
    prune_schedule's result, S the sequence length at the first level."""
    n_vis0 = levels[0]["token_group"].size
    lists = []
    for l in range(L):
        g = sum(1 for x in level_layer if x <= l)
        if g < len(levels):
            lists.append(np.asarray(levels[g]["keep_idx"], dtype=np.int32))
        else:
            kept_vis = int(levels[-1]["S_out"]) - (S - n_vis0)      # visual tokens the last level left
            lists.append(np.arange(S - n_vis0 + kept_vis, dtype=np.int32))
    return lists


# --------------------------------------------------------------------------- #
# a7 / a9: order-preserving row gathers
# --------------------------------------------------------------------------- #


def gather_rows(x: np.ndarray, keep_idx: np.ndarray) -> np.ndarray:
    out = np.empty((len(keep_idx),) + x.shape[1:], dtype=x.dtype)
    for i, src in enumerate(keep_idx):
        out[i] = x[src]
    return out


def prefill_prune(Q, K, hidden, vis_start, n_vis, token_group, group_budget, softmax_scale):
    """a5 + a6 + a7 chained, as the library's prefill call runs them."""
    S = K.shape[1]
    a = attention_scores(Q, K, vis_start, n_vis, softmax_scale)
    sel = weighted_topk(a, token_group, group_budget, S, vis_start)
    out = {"scores": a, "hidden_out": gather_rows(hidden, sel["keep_idx"])}
    out.update(sel)
    return out


# --------------------------------------------------------------------------- #
# a8 / a9: KV-cache selection and compaction ("Decoding: Prefilling-driven Optimization")
# --------------------------------------------------------------------------- #


def kv_select(policy: int, L: int, S_cur: int, vis_start: int, n_vis: int, l1: int = 0,
              keep_ratio: float = 1.0, scores: Optional[np.ndarray] = None,
              given: Optional[List[np.ndarray]] = None) -> List[np.ndarray]:
    """Per-layer ascending keep lists.

    PAPER: layers below l1 (0-based) keep every position; from l1 on, every
    visual position is dropped.  TOPK: each layer keeps the ceil(ratio*n_vis)
    best-scored visual tokens plus all non-visual positions.  GIVEN: the lists
    are the caller's.
    """
    if policy == KV_GIVEN:
        return [np.asarray(g, dtype=np.int32) for g in given]
    lists = []
    for layer in range(L):
        if policy == KV_PAPER:
            keep = np.ones(S_cur, dtype=bool)
            if layer >= l1:
                keep[vis_start:vis_start + n_vis] = False
            lists.append(np.nonzero(keep)[0].astype(np.int32))
        else:
            s = np.asarray(scores, dtype=np.float64)
            s = s[layer] if s.ndim == 2 else s
            budget = min(n_vis, ceilq(float(keep_ratio) * n_vis))
            sel = weighted_topk(s, np.zeros(n_vis, dtype=np.int32), [budget], S_cur, vis_start)
            lists.append(sel["keep_idx"])
    return lists


def kv_compact(k_layers: List[np.ndarray], v_layers: List[np.ndarray],
               keep_lists: List[np.ndarray]):
    """Out-of-place statement of the in-place gather: row i of every head's slab
    becomes the old row keep[i]; the new length is len(keep)."""
    new_k, new_v, new_len = [], [], []
    for Kl, Vl, keep in zip(k_layers, v_layers, keep_lists):
        new_k.append(np.stack([gather_rows(Kl[h], keep) for h in range(Kl.shape[0])]))
        new_v.append(np.stack([gather_rows(Vl[h], keep) for h in range(Vl.shape[0])]))
        new_len.append(len(keep))
    return new_k, new_v, np.asarray(new_len, dtype=np.int32)


def kv_bytes(keep_lists: List[np.ndarray], Hkv: int, dh: int, elem_bytes: int) -> int:
    """Bytes of K plus V held after compaction."""
    return int(sum(len(k) for k in keep_lists)) * 2 * Hkv * dh * elem_bytes

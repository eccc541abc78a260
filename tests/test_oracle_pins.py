"""Pins for the CPU oracle: what the paper and the mathematics fix, checked
without any GPU.  Each test is chosen so that a plausible slip in the oracle
(dropped term, wrong sign or index, transposed operand, off-by-one in a budget)
fails it.  The brute-force routines here are written with plain Python loops and
`math`, independently of the oracle's numpy code.
"""

import json
import math
import os

import numpy as np
import pytest
from scipy.special import softmax as scipy_softmax

from oracle import metok_oracle as O
from paper_2506_02850_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_constants.json")


# --------------------------------------------------------------------------- #
# independent brute force (pure Python)
# --------------------------------------------------------------------------- #


def py_cos(a, b):
    dot = sum(float(x) * float(y) for x, y in zip(a, b))
    na = max(math.sqrt(sum(float(x) ** 2 for x in a)), 1e-8)
    nb = max(math.sqrt(sum(float(x) ** 2 for x in b)), 1e-8)
    return dot / (na * nb)


def py_topk_desc(scores, n):
    """n best (score desc, index asc) by repeated scanning."""
    left = list(range(len(scores)))
    picked = []
    for _ in range(n):
        best = left[0]
        for j in left[1:]:
            if scores[j] > scores[best]:
                best = j
        picked.append(best)
        left.remove(best)
    return sorted(picked)


# --------------------------------------------------------------------------- #
# P1 / P2: planted events, closed forms (a1, a2)
# --------------------------------------------------------------------------- #


@pytest.mark.parametrize("name", ["tiny", "frames32", "frames64", "frames128d1024", "stress"])
def test_planted_boundaries_recovered(name):
    cfg = W.CONFIGS[name]
    vis = W.vision_inputs(cfg)
    for mode in (O.SIM_FLATTEN, O.SIM_MEANPOOL):
        if mode == O.SIM_MEANPOOL and (name == "stress" or cfg.near_dup):
            # averaging the tokens first leaves the 0.98 near-duplicate boundary
            # at ~0.9985, inside the spread of the within-event values
            continue
        seg = O.segment_events(vis["V"], cfg.k, mode)
        assert np.array_equal(seg["boundaries"], vis["boundaries"]), (name, mode)
        assert np.array_equal(seg["event_offsets"], vis["event_offsets"])
        assert seg["frame_event"][0] == 0 and seg["frame_event"][-1] == cfg.k - 1
        assert np.all(np.diff(seg["frame_event"]) >= 0)
        if mode == O.SIM_FLATTEN:
            sims = seg["sims"]
            inside = np.ones(cfg.T - 1, dtype=bool)
            inside[vis["boundaries"]] = False
            # E[cos] of two noisy copies of one base = 1 / (1 + sigma^2)
            assert abs(sims[inside].mean() - 1.0 / (1.0 + cfg.sigma ** 2)) < 2e-3
            cross = sims[~inside]
            if vis["near_dup_boundary"] is not None:
                b = vis["near_dup_boundary"]
                assert abs(sims[b] - 0.98) < 5e-3
                cross = np.delete(sims, np.concatenate([np.nonzero(inside)[0], [b]]))
            assert np.all(np.abs(cross) < 0.12)


def test_similarity_closed_forms():
    rng = np.random.default_rng(5)
    a = rng.standard_normal((3, 7))
    V = np.stack([a, a, 2.5 * a, -a])                      # cos = 1, 1, -1
    s = O.frame_similarity(V)
    assert np.allclose(s, [1.0, 1.0, -1.0], atol=1e-12)
    # orthogonal hand-built frames -> 0 ; 45 degrees -> 1/sqrt(2)
    e = np.zeros((3, 1, 4))
    e[0, 0, 0] = 1.0
    e[1, 0, 1] = 3.0
    e[2, 0, 1] = 1.0
    e[2, 0, 2] = 1.0
    s = O.frame_similarity(e)
    assert abs(s[0]) < 1e-15 and abs(s[1] - 1 / math.sqrt(2)) < 1e-12
    # FLATTEN and MEANPOOL differ: tokens that cancel in the mean
    V2 = np.zeros((2, 2, 2))
    V2[0] = [[1, 0], [0, 1]]
    V2[1] = [[0, 1], [1, 0]]                               # Frobenius dot 0, means equal
    assert abs(O.frame_similarity(V2, O.SIM_FLATTEN)[0]) < 1e-15
    assert abs(O.frame_similarity(V2, O.SIM_MEANPOOL)[0] - 1.0) < 1e-12
    # zero frame: clamped norm, finite result
    V3 = np.zeros((2, 2, 2))
    V3[1] = 1.0
    assert O.frame_similarity(V3)[0] == 0.0


def test_similarity_against_python_loops():
    rng = np.random.default_rng(6)
    V = rng.standard_normal((5, 3, 4))
    s = O.frame_similarity(V)
    for i in range(4):
        assert abs(s[i] - py_cos(V[i].ravel(), V[i + 1].ravel())) < 1e-12
    sm = O.frame_similarity(V, O.SIM_MEANPOOL)
    for i in range(4):
        assert abs(sm[i] - py_cos(V[i].mean(0), V[i + 1].mean(0))) < 1e-12


def test_split_events_ties_and_edges():
    sims = np.array([0.9, 0.1, 0.1, 0.8, 0.1])
    out = O.split_events(sims, 3)                          # two lowest, lower index first
    assert out["boundaries"].tolist() == [1, 2]
    assert out["event_offsets"].tolist() == [0, 2, 3, 6]
    assert out["frame_event"].tolist() == [0, 0, 1, 2, 2, 2]
    one = O.split_events(sims, 1)
    assert one["boundaries"].size == 0 and one["event_offsets"].tolist() == [0, 6]
    allk = O.split_events(sims, 6)
    assert allk["event_offsets"].tolist() == [0, 1, 2, 3, 4, 5, 6]


@pytest.mark.parametrize("name", ["tiny", "frames32", "frames64", "frames128d1024", "stress"])
def test_planted_relevant_events_become_key(name):
    cfg = W.CONFIGS[name]
    vis = W.vision_inputs(cfg)
    s = O.token_relevance(vis["V"], vis["t"])
    for agg in (O.AGG_MEAN, O.AGG_MAX):
        ev = O.key_events(s, cfg.T, cfg.N, vis["event_offsets"], cfg.alpha, agg)
        assert np.array_equal(np.nonzero(ev["event_is_key"])[0], vis["relevant_events"]), (name, agg)
    assert ev["event_is_key"].sum() == math.ceil(cfg.alpha * cfg.k)


def test_token_relevance_against_python_loops():
    rng = np.random.default_rng(7)
    V = rng.standard_normal((2, 3, 5))
    t = rng.standard_normal(5)
    s = O.token_relevance(V, t)
    X = V.reshape(-1, 5)
    for j in range(6):
        assert abs(s[j] - py_cos(X[j], t)) < 1e-12
    # scale invariance and sign
    assert np.allclose(O.token_relevance(3.0 * V, 0.5 * t), s, atol=1e-12)
    assert np.allclose(O.token_relevance(V, -t), -s, atol=1e-12)


def test_key_events_mean_vs_max_and_ties():
    # 3 events: frames [0,1], [2], [3,4,5]; N = 1
    ts = np.array([0.1, 0.9, 0.6, 0.5, 0.5, 0.5])
    offs = np.array([0, 2, 3, 6])
    mean = O.key_events(ts, 6, 1, offs, 0.5, O.AGG_MEAN)     # means .5 .6 .5 -> top 2 = {1, 0}
    assert np.allclose(mean["event_score"], [0.5, 0.6, 0.5])
    assert mean["event_is_key"].tolist() == [1, 1, 0]        # tie 0 vs 2 -> lower index
    mx = O.key_events(ts, 6, 1, offs, 0.5, O.AGG_MAX)        # max .9 .6 .5
    assert np.allclose(mx["event_score"], [0.9, 0.6, 0.5])
    assert mx["event_is_key"].tolist() == [1, 1, 0]
    one = O.key_events(ts, 6, 1, offs, 0.3, O.AGG_MAX)       # ceil(.9) = 1
    assert one["event_is_key"].tolist() == [1, 0, 0]


# --------------------------------------------------------------------------- #
# P6: constants the paper prints
# --------------------------------------------------------------------------- #


def test_printed_key_event_counts_and_schedule():
    g = json.load(open(GOLDEN))
    for hp in g["hyperparameters"]:
        want = g["key_event_counts"][str(hp["k"])]
        assert min(hp["k"], O.ceilq(hp["alpha"] * hp["k"])) == want
        ev = O.key_events(np.linspace(0, 1, hp["k"]), hp["k"], 1, np.arange(hp["k"] + 1), hp["alpha"])
        assert int(ev["event_is_key"].sum()) == want
    # r = 0.55, alpha = 0.5: Eq. 6 gives 1, r, r^2, 0 and Eq. 7 gives 1, alpha r, 0
    rk = [O.retention_ratios(0.5, 0.55, s) for s in range(4)]
    assert rk[0] == (1.0, 1.0)
    assert abs(rk[1][0] - 0.55) < 1e-7 and abs(rk[1][1] - 0.275) < 1e-7
    assert abs(rk[2][0] - 0.3025) < 1e-7 and rk[2][1] == 0.0
    assert rk[3] == (0.0, 0.0)
    r76 = O.retention_ratios(0.5, 0.76, 2)[0]
    assert abs(r76 - 0.5776) < 1e-6
    b = O.retention_budgets(0.5, 0.55, 1, (1000, 2000))
    assert b.tolist() == [550, 550]
    b = O.retention_budgets(0.5, 0.55, 2, (1000, 2000))
    assert b.tolist() == [303, 0]                          # ceil(302.5)
    assert O.retention_budgets(0.5, 0.55, 3, (1000, 2000)).tolist() == [0, 0]
    # exact products must not round up: 0.5 * 8 = 4, not 5
    assert O.ceilq(0.5 * 8) == 4
    assert O.ceilq(0.3 * 10) == 3 and O.ceilq(0.1 * 3 * 10) == 3   # 3.0000000000000004 is still 3
    assert O.ceilq(0.065 * 18432) == 1199 and O.ceilq(0.2 * 2304) == 461
    assert O.event_token_budget(10, 0.25) == 3 and O.event_token_budget(1, 0.01) == 1


def test_kv_policy_reproduces_printed_cache_sizes():
    """Table 3: with visual K/V kept only in layers 0..l1-1 (l1 = 3) and ~80 text
    tokens kept everywhere, the decode-stage cache is 22.3 / 171.8 of the
    stage-1 cache.  l1 = 2 or 4 (or 1-based layers) miss it by far."""
    g = json.load(open(GOLDEN))
    lay = g["kv_layout_7b"]
    per_tok = 2 * lay["kv_heads"] * lay["head_dim"] * lay["bytes_per_element"]
    mb = g["kv_cache_mb_llava_ov_7b"]
    tok_stage1 = mb["after_vision_encoding"] * 2 ** 20 / (per_tok * lay["layers"])
    n_text = 80
    n_vis = int(round(tok_stage1)) - n_text
    want = mb["after_decoding"] / mb["after_vision_encoding"]

    def ratio(l1):
        lists = O.kv_select(O.KV_PAPER, lay["layers"], n_vis + n_text, 0, n_vis, l1=l1)
        full = O.kv_select(O.KV_PAPER, lay["layers"], n_vis + n_text, 0, n_vis, l1=lay["layers"])
        return O.kv_bytes(lists, lay["kv_heads"], lay["head_dim"], 2) / O.kv_bytes(full, lay["kv_heads"], lay["head_dim"], 2)

    assert abs(ratio(3) - want) < 2e-3
    assert abs(ratio(2) - want) > 2e-2 and abs(ratio(4) - want) > 2e-2
    # absolute size in MiB too
    lists = O.kv_select(O.KV_PAPER, lay["layers"], n_vis + n_text, 0, n_vis, l1=3)
    assert abs(O.kv_bytes(lists, lay["kv_heads"], lay["head_dim"], 2) / 2 ** 20 - mb["after_decoding"]) < 0.3
    # Table 2's uncompressed LongVA cache = 128 x 144 visual tokens + ~79 others
    t2 = g["kv_cache_mb_table2"]
    tok = t2["longva_base"] * 2 ** 20 / (per_tok * lay["layers"])
    assert abs(tok - (128 * 144 + 79)) < 2


# --------------------------------------------------------------------------- #
# P3: brute force on tiny inputs (a3, a4, a6)
# --------------------------------------------------------------------------- #


@pytest.mark.parametrize("seed", range(6))
def test_key_token_topk_brute_force(seed):
    rng = np.random.default_rng(100 + seed)
    N = int(rng.integers(1, 5))
    lens = [int(v) for v in rng.integers(1, 5, size=int(rng.integers(1, 5)))]
    offs = np.concatenate([[0], np.cumsum(lens)])
    T = int(offs[-1])
    s = rng.standard_normal(T * N)
    s[rng.integers(0, T * N, size=T * N // 3)] = 0.25       # force ties
    is_key = rng.integers(0, 2, size=len(lens)).astype(np.uint8)
    kk, kn = 0.4, 0.2
    out = O.key_token_topk(s, N, offs, is_key, kk, kn)
    want = []
    for e, ln in enumerate(lens):
        lo, hi = offs[e] * N, offs[e + 1] * N
        m = hi - lo
        ratio = kk if is_key[e] else kn
        n = min(m, max(1, math.ceil(ratio * m - 1e-9)))
        assert out["event_budget"][e] == n
        want += [lo + j for j in py_topk_desc(list(s[lo:hi]), n)]
    assert out["key_idx"].tolist() == want
    assert out["is_key_token"].sum() == len(want)


@pytest.mark.parametrize("seed", range(6))
def test_merge_assign_brute_force(seed):
    rng = np.random.default_rng(200 + seed)
    N, d = 3, 5
    lens = [int(v) for v in rng.integers(1, 4, size=3)]
    offs = np.concatenate([[0], np.cumsum(lens)])
    T = int(offs[-1])
    V = rng.standard_normal((T, N, d))
    if seed % 2 == 0:
        V[1] = V[0]                                         # exact duplicate rows: tie -> lower key
    is_key = np.zeros(T * N, dtype=np.uint8)
    for e in range(3):
        lo, hi = offs[e] * N, offs[e + 1] * N
        pick = rng.choice(np.arange(lo, hi), size=max(1, (hi - lo) // 3), replace=False)
        is_key[pick] = 1
    out = O.merge_assign(V, N, offs, is_key, "f32")
    X = V.reshape(-1, d)
    keys = [j for j in range(T * N) if is_key[j]]
    slot = {j: i for i, j in enumerate(keys)}
    members = {i: [j] for j, i in slot.items()}
    for e in range(3):
        lo, hi = offs[e] * N, offs[e + 1] * N
        ek = [j for j in keys if lo <= j < hi]
        for a in range(lo, hi):
            if is_key[a]:
                assert out["assign"][a] == slot[a]
                continue
            best, best_c = None, -2.0
            for c in ek:                                     # ascending: strict > keeps lower c
                v = py_cos(X[a], X[c])
                if v > best_c + 0.0:
                    if best is None or v > best_c:
                        best, best_c = c, v
            assert out["assign"][a] == slot[best], (a, best)
            members[slot[best]].append(a)
    assert out["out_src"].tolist() == keys
    for i, js in members.items():
        mean = [sum(X[j][c] for j in js) / len(js) for c in range(d)]
        assert np.allclose(out["out_feats_exact"][i], mean, atol=1e-12)
        assert out["out_members"][i] == len(js)
        e = int(np.searchsorted(offs * N, keys[i], side="right") - 1)
        assert out["out_event"][i] == e


@pytest.mark.parametrize("seed", range(6))
def test_weighted_topk_brute_force(seed):
    rng = np.random.default_rng(300 + seed)
    n_vis, vis_start, Lt = 23, int(rng.integers(0, 4)), 3
    S = vis_start + n_vis + Lt
    s = np.round(rng.standard_normal(n_vis), 1)             # many ties
    grp = rng.integers(0, 3, size=n_vis).astype(np.int32)
    budget = [int(rng.integers(0, 12)) for _ in range(3)]
    out = O.weighted_topk(s, grp, budget, S, vis_start)
    keep = set(range(vis_start)) | set(range(vis_start + n_vis, S))
    for g in range(3):
        idx = [j for j in range(n_vis) if grp[j] == g]
        n = min(len(idx), budget[g])
        for r in py_topk_desc([s[j] for j in idx], n):
            keep.add(vis_start + idx[r])
    assert out["keep_idx"].tolist() == sorted(keep)
    assert out["S_out"] == len(keep)


# --------------------------------------------------------------------------- #
# P4: attention scores against textbook routines and closed forms (a5)
# --------------------------------------------------------------------------- #


def test_attention_scores_python_loops():
    rng = np.random.default_rng(8)
    Hq, Hkv, Lt, dh, S = 4, 2, 3, 5, 9
    Q = rng.standard_normal((Hq, Lt, dh))
    K = rng.standard_normal((Hkv, S, dh))
    vis_start, n_vis = 1, 4
    scale = 0.37
    got = O.attention_scores(Q, K, vis_start, n_vis, scale)
    sc = float(np.float32(scale))
    want = [0.0] * n_vis
    for h in range(Hq):
        g = h // 2
        for q in range(Lt):
            last = S - Lt + q
            lg = [sc * sum(Q[h, q, c] * K[g, u, c] for c in range(dh)) for u in range(last + 1)]
            z = sum(math.exp(v) for v in lg)
            for j in range(n_vis):
                want[j] += math.exp(lg[vis_start + j]) / z
    want = [w / (Hq * Lt) for w in want]
    assert np.allclose(got, want, rtol=1e-12, atol=0)


def test_attention_scores_vs_library_softmax_and_mass():
    rng = np.random.default_rng(9)
    Hq, Hkv, dh, S = 6, 3, 8, 40
    Q = rng.standard_normal((Hq, 1, dh))                    # Lt = 1: the query sees all S keys
    K = rng.standard_normal((Hkv, S, dh))
    sc = float(np.float32(dh ** -0.5))
    got = O.attention_scores(Q, K, 0, S - 1, dh ** -0.5)
    P = np.stack([scipy_softmax(sc * (K[h // 2] @ Q[h, 0])) for h in range(Hq)])
    assert np.allclose(got, P[:, : S - 1].mean(axis=0), rtol=1e-12)
    # total probability: visual mass + the text token's own mass = 1
    assert abs(got.sum() + P[:, S - 1].mean() - 1.0) < 1e-12
    # transposing the head grouping (h % Hkv instead of h // rep) must change the answer
    P_wrong = np.stack([scipy_softmax(sc * (K[h % 3] @ Q[h, 0])) for h in range(Hq)])
    assert not np.allclose(got, P_wrong[:, : S - 1].mean(axis=0), rtol=1e-3)


def test_attention_scores_closed_forms():
    Hq, Hkv, Lt, dh, S = 2, 1, 3, 4, 10
    K = np.ones((Hkv, S, dh))
    Q = np.ones((Hq, Lt, dh))
    # all logits equal: every visible key gets 1/#visible; query q sees S-Lt+q+1 keys
    got = O.attention_scores(Q, K, 0, S - Lt, 0.5)
    want = np.mean([1.0 / (S - Lt + q + 1) for q in range(Lt)])
    assert np.allclose(got, want, rtol=1e-13)
    # one key with a dominating logit takes all the mass, shifted logits do not overflow
    K2 = np.zeros((Hkv, S, dh))
    K2[0, 3] = 500.0
    got = O.attention_scores(Q, K2, 0, S - Lt, 1.0)
    assert abs(got[3] - 1.0) < 1e-12 and abs(got.sum() - 1.0) < 1e-12
    # a later text token is invisible to earlier queries: key S-1 only to the last query
    K3 = np.zeros((Hkv, S, dh))
    K3[0, S - 1] = 500.0
    got = O.attention_scores(Q, K3, 0, S - Lt, 1.0)
    q_see = [1.0 / (S - Lt + q + 1) for q in range(Lt - 1)] + [0.0]
    assert np.allclose(got, np.mean(q_see), rtol=1e-12)


# --------------------------------------------------------------------------- #
# P5: invariants on a mid-size random case and on the tiny config
# --------------------------------------------------------------------------- #


def test_compress_vision_invariants():
    cfg = W.CONFIGS["frames32"]
    vis = W.vision_inputs(cfg)
    V = vis["V"][:12, :36]                                   # 12 frames x 36 tokens
    offs = np.array([0, 3, 4, 9, 12])
    out = O.compress_vision(V, vis["t"], offs, 0.5, 0.3, 0.1, "bf16")
    T, N, d = V.shape
    X = V.reshape(-1, d).astype(np.float64)
    n_out = out["n_out"]
    assert n_out == int(out["event_budget"].sum()) == out["key_idx"].size
    assert out["out_members"].sum() == T * N and out["out_members"].min() >= 1
    assert np.all(np.diff(out["out_src"]) > 0)
    tok_event = np.repeat(np.searchsorted(offs, np.arange(T), side="right") - 1, N)
    assert np.array_equal(out["out_event"][out["assign"]], tok_event)       # stays in its own event
    assert np.array_equal(out["assign"][out["out_src"]], np.arange(n_out))
    for e in range(4):                                        # mass conservation per event
        sl = out["out_event"] == e
        lhs = (out["out_members"][sl, None] * out["out_feats_exact"][sl]).sum(axis=0)
        assert np.allclose(lhs, X[tok_event == e].sum(axis=0), atol=1e-9)
    for c in range(n_out):                                    # convex combination
        mem = X[out["assign"] == c]
        assert np.all(out["out_feats_exact"][c] <= mem.max(axis=0) + 1e-12)
        assert np.all(out["out_feats_exact"][c] >= mem.min(axis=0) - 1e-12)
    # output rounding: representable in bf16 and within half an ulp
    r = out["out_feats"]
    assert np.array_equal(W.round_to_bf16(r.astype(np.float32)).astype(np.float64), r)
    assert np.all(np.abs(r - out["out_feats_exact"]) <= np.abs(out["out_feats_exact"]) * 2.0 ** -8 + 1e-300)


def test_round_bf16_matches_bit_level_rounding():
    rng = np.random.default_rng(11)
    x = rng.standard_normal(20000).astype(np.float32) * np.float32(3.0)
    x[:4] = [1.00390625, 1.01171875, -1.00390625, 0.0]        # exact ties -> even
    assert np.array_equal(O.round_bf16(x.astype(np.float64)), W.round_to_bf16(x).astype(np.float64))


def test_keep_ratio_one_is_identity_and_k1():
    cfg = W.CONFIGS["tiny"]
    vis = W.vision_inputs(cfg)
    seg = O.segment_events(vis["V"], 1)
    assert seg["event_offsets"].tolist() == [0, cfg.T]
    out = O.compress_vision(vis["V"], vis["t"], seg["event_offsets"], 0.5, 1.0, 1.0, "f32")
    assert out["n_out"] == cfg.Nv and np.all(out["out_members"] == 1)
    assert np.array_equal(out["assign"], np.arange(cfg.Nv))
    assert np.array_equal(out["out_feats"], vis["V"].reshape(cfg.Nv, cfg.d).astype(np.float64))


def test_prefill_prune_invariants_and_budget_zero():
    cfg = W.CONFIGS["tiny"]
    vis = W.vision_inputs(cfg)
    grp = W.token_groups(cfg, cfg.Nv, vis=vis)
    pf = W.prefill_inputs(cfg, 1, cfg.Nv, grp, vis_start=2)
    S = pf["S"]
    hidden = W.payload_rows_np(W.hidden_salt(cfg, 1), np.arange(S), cfg.D, "f32")
    N0 = [int((grp == 0).sum()), int((grp == 1).sum())]
    for stage in (1, 2, 3):
        b = O.retention_budgets(cfg.alpha, cfg.keep_prefill, stage, N0)
        out = O.prefill_prune(pf["Q"], pf["K"], hidden, 2, cfg.Nv, grp, b, cfg.dh ** -0.5)
        keep = out["keep_idx"]
        assert np.all(np.diff(keep) > 0)
        assert out["S_out"] == 2 + cfg.Lt + int(b.sum())       # survivors = the schedule's budget
        assert set(range(2)) <= set(keep.tolist()) and set(range(S - cfg.Lt, S)) <= set(keep.tolist())
        kept_vis = keep[(keep >= 2) & (keep < 2 + cfg.Nv)] - 2
        for g in (0, 1):
            assert int((grp[kept_vis] == g).sum()) == b[g]
        assert np.array_equal(out["hidden_out"], hidden[keep])
        if stage == 3:
            assert kept_vis.size == 0
    # every kept visual token of a class scores at least as high as every dropped one of that class
    b = O.retention_budgets(cfg.alpha, cfg.keep_prefill, 1, N0)
    out = O.prefill_prune(pf["Q"], pf["K"], hidden, 2, cfg.Nv, grp, b, cfg.dh ** -0.5)
    kept = np.zeros(cfg.Nv, dtype=bool)
    kv = out["keep_idx"][(out["keep_idx"] >= 2) & (out["keep_idx"] < 2 + cfg.Nv)] - 2
    kept[kv] = True
    for g in (0, 1):
        m = grp == g
        assert out["scores"][m & kept].min() >= out["scores"][m & ~kept].max()


def test_planted_relevance_separates_classes():
    """The planted rank-1 component must make attention scores informative:
    key-event tokens score higher on average, and the spread is far outside the
    near-tie band (otherwise index parity would test nothing)."""
    cfg = W.CONFIGS["frames32"]
    n_vis = 600
    grp = W.token_groups(cfg, n_vis, n_key=300)
    pf = W.prefill_inputs(cfg, 1, n_vis, grp)
    a = O.attention_scores(pf["Q"], pf["K"], 0, n_vis, cfg.dh ** -0.5)
    assert a[grp == 0].mean() > 1.5 * a[grp == 1].mean()
    assert a.std() / a.mean() > 0.5
    flat = W.prefill_inputs(cfg, 1, n_vis, grp, planted=False)
    a0 = O.attention_scores(flat["Q"], flat["K"], 0, n_vis, cfg.dh ** -0.5)
    assert a0.std() / a0.mean() < 0.2


# --------------------------------------------------------------------------- #
# a8 / a9: KV selection and compaction
# --------------------------------------------------------------------------- #


def test_kv_policies_and_compaction():
    cfg = W.CONFIGS["tiny"]
    L, Hkv, S, dh = 3, 2, 20, 4
    n_vis, vis_start = 14, 2
    rng = np.random.default_rng(12)
    ks = [rng.integers(0, 1000, size=(Hkv, S, dh)).astype(np.float32) for _ in range(L)]
    vs = [rng.integers(0, 1000, size=(Hkv, S, dh)).astype(np.float32) for _ in range(L)]
    paper = O.kv_select(O.KV_PAPER, L, S, vis_start, n_vis, l1=1)
    assert paper[0].tolist() == list(range(S))
    assert paper[1].tolist() == [0, 1, 16, 17, 18, 19] == paper[2].tolist()
    sc = rng.standard_normal((L, n_vis))
    topk = O.kv_select(O.KV_TOPK, L, S, vis_start, n_vis, keep_ratio=0.3, scores=sc)
    for layer in range(L):
        want = sorted([0, 1, 16, 17, 18, 19] + [vis_start + j for j in py_topk_desc(list(sc[layer]), 5)])
        assert topk[layer].tolist() == want                    # ceil(0.3*14) = 5
    shared = O.kv_select(O.KV_TOPK, L, S, vis_start, n_vis, keep_ratio=0.3, scores=sc[0])
    assert all(np.array_equal(s_, topk[0]) for s_ in shared)
    nk, nv, nl = O.kv_compact(ks, vs, topk)
    assert nl.tolist() == [11, 11, 11]
    for layer in range(L):
        for h in range(Hkv):
            for i, src in enumerate(topk[layer]):
                assert np.array_equal(nk[layer][h, i], ks[layer][h, src])
                assert np.array_equal(nv[layer][h, i], vs[layer][h, src])
    # no text rows at all (the tiny configuration's cache): only visual survivors remain
    only = O.kv_select(O.KV_TOPK, 1, n_vis, 0, n_vis, keep_ratio=0.5, scores=sc[0])
    assert len(only[0]) == 7
    none = O.kv_select(O.KV_PAPER, 1, n_vis, 0, n_vis, l1=0)
    assert len(none[0]) == 0
    assert O.kv_bytes(topk, Hkv, dh, 2) == 33 * 2 * Hkv * dh * 2


# --------------------------------------------------------------------------- #
# the paper's own stage-1 compressor: key frames and adaptive pooling
# --------------------------------------------------------------------------- #


def test_pool2d_and_adaptive_pool():
    g = np.arange(16, dtype=np.float64).reshape(16, 1)          # 4x4 grid, d = 1
    p = O.pool2d(g, 4, 2)
    assert p.ravel().tolist() == [2.5, 4.5, 10.5, 12.5]
    p3 = O.pool2d(g, 4, 3)                                       # clipped edge windows
    assert p3.shape == (4, 1)
    assert p3.ravel().tolist() == [5.0, 7.0, 13.0, 15.0]
    assert O.pool2d(g, 4, 1).ravel().tolist() == list(range(16))
    # divisible grid conserves the frame mean
    rng = np.random.default_rng(13)
    f = rng.standard_normal((144, 3))
    for s in (2, 3, 4, 6):
        assert np.allclose(O.pool2d(f, 12, s).mean(axis=0), f.mean(axis=0), atol=1e-12)
    # key frames: ceil(beta * len) best per event
    fs = np.array([.1, .5, .3, .9, .2, .2, .2])
    kf = O.key_frames(fs, np.array([0, 3, 7]), 0.4)              # ceil(1.2)=2 of 3 ; ceil(1.6)=2 of 4
    assert kf.tolist() == [0, 1, 1, 1, 1, 0, 0]
    # strides (2,3) in key events become (4,6) in non-key events with alpha = 0.5
    cfg = W.CONFIGS["frames32"]
    vis = W.vision_inputs(cfg)
    out = O.adaptive_pool(vis["V"][:, :, :32], vis["t"][:32], vis["event_offsets"], 0.5, 0.45,
                          (2, 3, 4, 6), "bf16")
    per = {2: 36, 3: 16, 4: 9, 6: 4}
    assert out["n_out"] == sum(per[int(s)] for s in out["frame_stride"])
    assert np.all(np.diff(out["out_frame"]) >= 0)
    ek = np.repeat(out["event_is_key"], np.diff(vis["event_offsets"]))
    assert set(out["frame_stride"][ek == 1]) <= {2, 3} and set(out["frame_stride"][ek == 0]) <= {4, 6}


def test_prune_schedule_planted_order_and_printed_ratios():
    """Three levels on logits planted per level (one head, one text query, K[j] = c_j u, Q = u, so
    the score is monotone in c_j): the survivors must be the per-class top budgets of a plain sort
    of c, with the paper's r = 0.55, alpha = 0.5 (stage ratios .55/.275, .3025/0, 0/0)."""
    rng = np.random.default_rng(11)
    dh, n_vis, vis_start, tail = 8, 300, 3, 2                  # 2 non-visual positions after the visual span, 1 text query last
    group = (rng.random(n_vis) < 0.33).astype(np.int32)       # 1 = non-key
    N0 = [int((group == 0).sum()), int((group == 1).sum())]
    u = np.zeros(dh); u[2] = 1.0
    alive = np.arange(n_vis)
    Qs, Ks, want_alive, cs = [], [], [], []
    for stage, ratios in zip((1, 2, 3), ((0.55, 0.275), (0.3025, 0.0), (0.0, 0.0))):
        c = rng.permutation(alive.size).astype(np.float64) * 0.01      # distinct, reshuffled at every level
        S = vis_start + alive.size + tail + 1
        K = rng.standard_normal((1, S, dh)) * 0.01
        K[0, :, 2] = 0.0
        K[0, vis_start:vis_start + alive.size] += c[:, None] * u[None, :]
        Qs.append(u[None, None, :].copy()); Ks.append(K); cs.append(c)
        keep = []
        for g in (0, 1):
            members = [i for i in range(alive.size) if group[alive[i]] == g]
            n = min(len(members), math.ceil(ratios[g] * N0[g] - 1e-9))
            keep += sorted(members, key=lambda i: -c[i])[:n]
        alive = alive[sorted(keep)]
        want_alive.append(alive)
    lv = O.prune_schedule(Qs, Ks, group, 0.5, 0.55, vis_start, 1.0)
    assert len(lv) == 3
    assert lv[0]["budget"].tolist() == [math.ceil(0.55 * N0[0] - 1e-9), math.ceil(0.275 * N0[1] - 1e-9)]
    for s in range(3):
        S = Ks[s].shape[1]
        n_in = lv[s]["token_group"].size
        k = lv[s]["keep_idx"]
        vis = k[(k >= vis_start) & (k < vis_start + n_in)] - vis_start
        assert np.array_equal(lv[s]["origin"][vis], want_alive[s]), s
        assert np.array_equal(lv[s]["token_group"], group[lv[s]["origin"]])
        non_vis = [p for p in range(S) if not (vis_start <= p < vis_start + n_in)]
        assert set(non_vis) <= set(k.tolist())                 # every non-visual position survives
    assert want_alive[1].size == math.ceil(0.3025 * N0[0] - 1e-9) and want_alive[2].size == 0
    assert np.all(group[want_alive[1]] == 0)                   # no non-key token passes the second level


def test_given_key_events_replace_the_scored_ones():
    """The random-key-event ablation: a caller's key-event mask only changes which per-event ratio
    applies (brute-force count of the budgets), and the scored mask given back reproduces the default."""
    rng = np.random.default_rng(21)
    T, N, d = 9, 16, 12
    offs = np.array([0, 2, 5, 9], dtype=np.int32)
    V = rng.standard_normal((T, N, d))
    t = rng.standard_normal(d)
    base = O.compress_vision(V, t, offs, 0.5, 0.5, 0.1, "f32")
    same = O.compress_vision(V, t, offs, 0.5, 0.5, 0.1, "f32", key_events_given=base["event_is_key"])
    assert np.array_equal(base["out_src"], same["out_src"]) and np.array_equal(base["assign"], same["assign"])
    flipped = ~base["event_is_key"].astype(bool)
    other = O.compress_vision(V, t, offs, 0.5, 0.5, 0.1, "f32", key_events_given=flipped)
    assert np.array_equal(other["event_is_key"].astype(bool), flipped)
    want = sum(max(1, math.ceil((0.5 if flipped[e] else 0.1) * (offs[e + 1] - offs[e]) * N - 1e-9)) for e in range(3))
    assert other["n_out"] == want and other["n_out"] != base["n_out"]
    assert np.array_equal(other["token_score"], base["token_score"])          # the scores themselves do not change


def test_near_threshold_band_members_known_by_construction():
    """The band that excuses a top-k mismatch is |s - tau| < 1e-3 * max(|tau|, 1e-3 * max|s|).
    Hand-built vectors whose band members are known: a band ten times too wide, a band taken
    relative to the largest score instead of the threshold, or a missing floor each fail."""
    # threshold 1.0: 1 +- 5e-4 inside, 1 +- 2e-3 outside, and the threshold itself inside
    s = np.array([50.0, 1.002, 1.0005, 1.0, 0.9995, 0.998, -1.0, 0.0])
    assert O.near_threshold(s, 1.0).tolist() == [False, False, True, True, True, False, False, False]
    # relative to |tau|, not to max|s| = 50 (that band would be 5e-2 wide and take in 1.002 and 0.998)
    assert O.near_threshold(s, 1.0).sum() == 3
    # a negative threshold uses its magnitude
    assert O.near_threshold(np.array([-2.0, -2.001, -2.003, 2.0]), -2.0).tolist() == [True, True, False, False]
    # threshold near zero: the band is floored at 1e-3 * 1e-3 * max|s| = 4e-6 here
    s0 = np.array([4.0, 1e-7, 3e-6, -3e-6, 5e-6, -5e-6, 0.0])
    assert O.near_threshold(s0, 0.0).tolist() == [False, True, True, True, False, False, True]
    assert O.near_threshold(s0, 1e-7).tolist() == [False, True, True, True, False, False, True]
    # just inside and just outside one band width (1.024 at a threshold of 1024)
    assert O.near_threshold(np.array([1024.0, 1025.0, 1025.05, 1022.95]), 1024.0).tolist() == [True, True, False, False]
    # width scales with the threshold: the same absolute gap is inside at 100, outside at 1
    assert O.near_threshold(np.array([100.0, 100.05]), 100.0).tolist() == [True, True]
    assert O.near_threshold(np.array([1.0, 1.05]), 1.0).tolist() == [True, False]
    assert O.NEAR_TIE == 1e-3


def test_key_token_and_class_topk_report_the_band_of_their_own_threshold():
    """key_token_topk and weighted_topk must hand near_threshold the LAST KEPT score of the segment
    or class (not the first dropped one, not another segment's)."""
    # one event of 8 tokens, budget 4: kept {10, 9, 8, 7.001}; 7.0 is dropped, 0.07 % below the cut
    ts = np.array([10.0, 9.0, 8.0, 7.001, 7.0, 6.9, 1.0, 0.5])
    out = O.key_token_topk(ts, 8, np.array([0, 1]), np.array([1], dtype=np.uint8), 0.5, 0.5)
    assert out["key_idx"].tolist() == [0, 1, 2, 3]
    assert out["near_tie"].tolist() == [False, False, False, True, True, False, False, False]
    # two classes with their own cuts: class 0 cut at 5.0 (4.998 near, 4.9 not), class 1 cut at 0.5
    sc = np.array([9.0, 5.0, 4.998, 4.9, 0.9, 0.5, 0.5004, 0.2])
    grp = np.array([0, 0, 0, 0, 1, 1, 1, 1])
    w = O.weighted_topk(sc, grp, [2, 3], 8, 0)
    assert w["keep_idx"].tolist() == [0, 1, 4, 5, 6]
    assert w["near_tie"].tolist() == [False, True, True, False, False, True, True, False]


def test_merge_margin_closed_form():
    """margin = (best - second best cosine) / |best| over the keys of the token's own event.
    Three keys at known angles from a non-key token: cosines cos(10 deg), cos(20 deg), cos(60 deg) by
    construction, so the margin is known in closed form; a margin taken from the wrong two
    columns (best vs worst, second vs third) or divided by the second gives another number."""
    def unit(deg):
        return np.array([math.cos(math.radians(deg)), math.sin(math.radians(deg)), 0.0, 0.0])
    a = unit(0.0) * 3.0                                     # the non-key token (norm must not matter)
    k1, k2, k3 = unit(60.0) * 0.5, unit(10.0) * 2.0, unit(-20.0) * 7.0
    # event 0: tokens a, k1, k2, k3; event 1: a copy of a whose only key is far away (one key: margin inf)
    V = np.stack([a, k1, k2, k3, a, unit(90.0)]).reshape(6, 1, 4)
    offs = np.array([0, 4, 6])
    is_key = np.array([0, 1, 1, 1, 0, 1], dtype=np.uint8)
    out = O.merge_assign(V, 1, offs, is_key, "f32")
    c10, c20, c60 = (math.cos(math.radians(x)) for x in (10.0, 20.0, 60.0))
    assert out["assign"][0] == 1                            # slot of k2 (the 10-degree key)
    assert math.isclose(out["margin"][0], (c10 - c20) / c10, rel_tol=1e-12)
    assert abs(out["margin"][0] - (c10 - c60) / c10) > 0.3   # not best-vs-worst
    assert math.isinf(out["margin"][4]) and out["assign"][4] == 3
    assert all(math.isinf(out["margin"][j]) for j in (1, 2, 3, 5))     # key tokens decide nothing
    # near-tie by construction: second key 1e-4 (relative) below the best -> inside the 1e-3 band;
    # 1e-2 below -> outside
    for rel, inside in ((1e-4, True), (1e-2, False)):
        ang = math.degrees(math.acos(c10 * (1.0 - rel)))
        V2 = np.stack([a, unit(10.0), unit(-ang)]).reshape(3, 1, 4)
        o2 = O.merge_assign(V2, 1, np.array([0, 3]), np.array([0, 1, 1], dtype=np.uint8), "f32")
        assert math.isclose(o2["margin"][0], rel, rel_tol=1e-6)
        assert (o2["margin"][0] < O.NEAR_TIE) == inside
    # negative best cosine: the margin divides by its magnitude and stays positive
    V3 = np.stack([a, unit(120.0), unit(150.0)]).reshape(3, 1, 4)
    o3 = O.merge_assign(V3, 1, np.array([0, 3]), np.array([0, 1, 1], dtype=np.uint8), "f32")
    c120, c150 = math.cos(math.radians(120.0)), math.cos(math.radians(150.0))
    assert o3["assign"][0] == 0 and math.isclose(o3["margin"][0], (c120 - c150) / abs(c120), rel_tol=1e-12)


def test_split_events_non_finite_similarity_ranks_last():
    """A frame with a non-finite feature gives NaN similarities on both sides; they count as the
    LARGEST values (never a boundary while finite candidates remain), ties to the lower index."""
    sims = np.array([0.9, 0.1, np.nan, np.nan, 0.5, 0.2, 0.95])
    assert O.split_events(sims, 3)["boundaries"].tolist() == [1, 5]
    assert O.split_events(sims, 6)["boundaries"].tolist() == [0, 1, 4, 5, 6]
    assert O.split_events(sims, 7)["boundaries"].tolist() == [0, 1, 2, 4, 5, 6]     # then the lower NaN
    V = np.random.default_rng(3).standard_normal((6, 2, 4))
    V[3, 1, 2] = np.inf
    out = O.segment_events(V, 3)
    assert np.isnan(out["sims"][2]) and np.isnan(out["sims"][3]) and np.isfinite(out["sims"][[0, 1, 4]]).all()
    assert not set(out["boundaries"].tolist()) & {2, 3}


def test_given_key_frames_replace_the_scored_ones():
    """The random-key-frame ablation of Algorithm 1: a caller's key-frame mask only changes which stride
    a frame is pooled with (output sizes counted by hand), and the scored mask given back reproduces
    the default."""
    rng = np.random.default_rng(23)
    T, G, d = 7, 6, 5
    offs = np.array([0, 3, 7], dtype=np.int32)
    V = rng.standard_normal((T, G * G, d))
    t = rng.standard_normal(d)
    strides = (1, 2, 3, 6)
    base = O.adaptive_pool(V, t, offs, 0.5, 0.5, strides, "f32")
    same = O.adaptive_pool(V, t, offs, 0.5, 0.5, strides, "f32", key_frames_given=base["frame_is_key"])
    assert np.array_equal(base["out_feats"], same["out_feats"]) and np.array_equal(base["out_frame"], same["out_frame"])
    given = np.array([1, 0, 0, 0, 0, 1, 1], dtype=np.uint8)
    out = O.adaptive_pool(V, t, offs, 0.5, 0.5, strides, "f32", key_frames_given=given)
    assert np.array_equal(out["frame_is_key"], given)
    want_stride = [(strides[0] if given[f] else strides[1]) if out["event_is_key"][0 if f < 3 else 1]
                   else (strides[2] if given[f] else strides[3]) for f in range(T)]
    assert out["frame_stride"].tolist() == want_stride
    assert out["n_out"] == sum((-(-G // s_)) ** 2 for s_ in want_stride)
    assert np.array_equal(out["event_is_key"], base["event_is_key"])            # the events' classes do not change
    f = 5                                                                       # a frame pooled with its given stride
    lo = int(np.searchsorted(out["out_frame"], f))
    assert np.allclose(out["out_feats_exact"][lo:lo + (-(-G // want_stride[f])) ** 2], O.pool2d(V[f], G, want_stride[f]))


def test_schedule_kv_lists_by_construction():
    """Layer groups and their lists, hand-built: 6 visual + 2 text positions, pruning layers 2 and 5 of 7."""
    lv1 = {"keep_idx": np.array([0, 2, 3, 5, 6, 7], dtype=np.int32), "S_out": 6, "token_group": np.zeros(6, dtype=np.int32)}
    lv2 = {"keep_idx": np.array([1, 4, 5], dtype=np.int32), "S_out": 3, "token_group": np.zeros(4, dtype=np.int32)}
    lists = O.schedule_kv_lists([lv1, lv2], [2, 5], 7, 8)
    assert [l.tolist() for l in lists[:2]] == [[0, 2, 3, 5, 6, 7]] * 2            # before the first pruning layer: what level 1 keeps
    assert [l.tolist() for l in lists[2:5]] == [[1, 4, 5]] * 3                    # between the two: what level 2 keeps, in level 2's layout
    assert [l.tolist() for l in lists[5:]] == [[0, 1, 2]] * 2                     # from the last pruning layer on: all rows that are left
    # a real chain: every list is ascending, inside its layer's cache, and text positions always survive
    rng = np.random.default_rng(8)
    n_vis, Lt, Hq, dh = 40, 3, 2, 8
    group = (rng.random(n_vis) < 0.5).astype(np.int32)
    Qs, Ks, g = [], [], group
    N0 = [int((group == 0).sum()), int((group == 1).sum())]
    for s_ in range(1, 4):
        Qs.append(rng.standard_normal((Hq, Lt, dh))); Ks.append(rng.standard_normal((1, g.size + Lt, dh)))
        lv = O.prune_schedule(Qs, Ks, group, 0.5, 0.6, 0, 0.3)
        k_ = lv[-1]["keep_idx"]
        g = g[k_[k_ < g.size]]
    lists = O.schedule_kv_lists(lv, [1, 2, 4], 6, n_vis + Lt)
    sizes = [n_vis + Lt] + [int(x["S_out"]) for x in lv]
    for l, lst in enumerate(lists):
        grp = sum(1 for x in (1, 2, 4) if x <= l)
        assert np.all(np.diff(lst) > 0) and lst[-1] < sizes[grp]
        assert lst[-Lt:].tolist() == list(range(sizes[grp] - Lt, sizes[grp]))
        assert lst.size == sizes[min(grp + 1, 3)]

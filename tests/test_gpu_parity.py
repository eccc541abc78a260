"""CUDA path vs CPU oracle through the C ABI, on the seeded workloads and on edge
cases.  Index outputs bit-exact outside the 1e-3 near-tie band; scores and
features within 2e-2 (bf16) / 1e-5 (fp32); gathers bit-exact."""

import math

import numpy as np
import pytest
import torch

from oracle import metok_oracle as O
from paper_2506_02850_b200 import binding as B
from paper_2506_02850_b200 import workloads as W
from tests import parity as P
from tests import runners as R

pytestmark = pytest.mark.gpu

MAX_ASSIGN_FLIPS = 8        # merge assignments that may differ from the oracle's inside the near-tie band
_vis_cache = {}


def vis_of(name):
    if name not in _vis_cache:
        _vis_cache.clear()                                     # the large ones are several hundred MB
        _vis_cache[name] = W.vision_inputs(W.CONFIGS[name])
    return _vis_cache[name]


# ------------------------------------------------------------------ a1 ----- #

@pytest.mark.parametrize("name", ["tiny", "frames32", "frames64", "frames128", "frames128d1024", "stress"])
def test_segment_events_workloads(name):
    cfg = W.CONFIGS[name]
    vis = vis_of(name)
    rep = R.segment_case(vis["V"], cfg.dtype, cfg.k, O.SIM_FLATTEN)
    assert rep["mismatches"] == 0
    got = B.metok_segment_events(P.to_torch(vis["V"], cfg.dtype), cfg.k)
    assert np.array_equal(got["boundaries"].cpu().numpy(), vis["boundaries"])   # the planted events


@pytest.mark.parametrize("name", ["tiny", "frames32", "frames128d1024"])
def test_segment_events_meanpool(name):
    cfg = W.CONFIGS[name]
    rep = R.segment_case(vis_of(name)["V"], cfg.dtype, cfg.k, O.SIM_MEANPOOL)
    assert rep["mismatches"] == 0


@pytest.mark.parametrize("T,N,d,k,dtype", [
    (1, 3, 8, 1, "bf16"), (2, 1, 8, 2, "bf16"), (3, 5, 72, 2, "f32"), (9, 7, 40, 9, "bf16"),
    (17, 33, 200, 5, "bf16"), (40, 130, 264, 1, "f32"), (5, 1030, 1032, 3, "bf16"), (700, 2, 16, 350, "f32")])
def test_segment_events_ragged(T, N, d, k, dtype):
    rng = np.random.default_rng(T * 1000 + N)
    V = W.quantize(rng.standard_normal((T, N, d)).astype(np.float32), dtype)
    for mode in (O.SIM_FLATTEN, O.SIM_MEANPOOL):
        R.segment_case(V, dtype, k, mode)


def test_segment_events_ties_go_to_lower_index_and_repeatable():
    base = np.random.default_rng(3).standard_normal((4, 16)).astype(np.float32)
    V = np.stack([base, base, base, base, -base, -base])      # sims 1,1,1,-1,1 ; ties among the 1s
    got = B.metok_segment_events(P.to_torch(V, "f32"), 4)
    assert got["boundaries"].cpu().tolist() == [0, 1, 3]      # the -1, then the two lowest-index ties
    vis = vis_of("frames32")
    x = P.to_torch(vis["V"], "bf16")
    a = B.metok_segment_events(x, 4)["sims"].clone()
    for _ in range(5):
        assert torch.equal(a, B.metok_segment_events(x, 4)["sims"])


@pytest.mark.parametrize("dtype,bad", [("f32", float("inf")), ("f32", float("nan")), ("bf16", float("inf"))])
def test_segment_events_non_finite_frame_still_gives_k_minus_1_boundaries(dtype, bad):
    """One frame holds a non-finite feature: its two similarities are NaN, rank as the largest, and
    exactly k-1 boundaries are written (none of them stale)."""
    rng = np.random.default_rng(17)
    T, N, d, k = 12, 8, 64, 4
    V = W.quantize(rng.standard_normal((T, N, d)).astype(np.float32), dtype).astype(np.float64)
    V[5, 3, 7] = bad
    want = O.segment_events(V, k)
    t = torch.from_numpy(V.astype(np.float32))
    t = (t.to(torch.bfloat16) if dtype == "bf16" else t).cuda()
    for call in (B.metok_segment_events, B.metok_segment_events_static):
        got = call(t, k)
        torch.cuda.synchronize()
        s = got["sims"].cpu().numpy()
        assert np.isnan(s[4]) and np.isnan(s[5]) and np.isfinite(np.delete(s, [4, 5])).all()
        assert np.array_equal(got["boundaries"].cpu().numpy(), want["boundaries"])
        assert np.array_equal(got["event_offsets"].cpu().numpy(), want["event_offsets"])
        assert np.array_equal(got["frame_event"].cpu().numpy(), want["frame_event"])


@pytest.mark.parametrize("name", ["tiny", "frames32", "frames64", "frames128", "frames128d1024", "stress"])
def test_segment_score_events_one_pass(name):
    """Segmentation and Eq. 5 token scores from one pass over V: both against the oracle, and the
    compressor fed with them against the compressor that scores by itself."""
    cfg = W.CONFIGS[name]
    vis = vis_of(name)
    Vd, td = P.to_torch(vis["V"], cfg.dtype), P.to_torch(vis["t"], cfg.dtype)
    got = B.metok_segment_score_events(Vd, cfg.k, td)
    want = O.segment_events(vis["V"], cfg.k)
    P.check_scores(got["sims"].cpu().numpy(), want["sims"], cfg.dtype, "sims")
    assert np.array_equal(got["boundaries"].cpu().numpy(), want["boundaries"])
    assert np.array_equal(got["event_offsets"].cpu().numpy(), want["event_offsets"])
    assert np.array_equal(got["frame_event"].cpu().numpy(), want["frame_event"])
    ts = O.token_relevance(vis["V"], vis["t"])
    P.check_scores(got["token_score"].cpu().numpy(), ts, cfg.dtype, "token_score")
    norms = np.sqrt((vis["V"].reshape(cfg.Nv, -1).astype(np.float64) ** 2).sum(axis=1))
    assert np.allclose(got["token_inv_norm"].cpu().numpy(), 1.0 / np.maximum(norms, 1e-8), rtol=1e-5)
    p = B.vision_params(cfg.alpha, cfg.keep_enc, cfg.keep_enc)
    a = B.metok_compress_vision(Vd, got["event_offsets"], td, p)
    b = B.metok_compress_vision(Vd, got["event_offsets"], td, p, scored=got)
    torch.cuda.synchronize()
    n = int(a["n_out"].item())
    assert n == int(b["n_out"].item())
    assert np.array_equal(a["event_is_key"].cpu().numpy(), b["event_is_key"].cpu().numpy())
    same = float(np.mean(a["out_src"][:n].cpu().numpy() == b["out_src"][:n].cpu().numpy()))
    assert same > 0.995, same                                  # the two scoring passes round differently in near-ties
    want_c = O.compress_vision(vis["V"], vis["t"], want["event_offsets"], cfg.alpha, cfg.keep_enc, cfg.keep_enc, cfg.dtype)
    P.check_index_set(b["out_src"][:n].cpu().numpy(), want_c["out_src"], lambda j: bool(want_c["near_tie"][j]),
                      "key tokens from one-pass scores")


def test_segment_score_events_ragged():
    for T, N, d, k, dtype in [(3, 5, 72, 2, "f32"), (9, 7, 40, 9, "bf16"), (17, 33, 264, 5, "bf16"), (5, 3, 2056, 3, "bf16")]:
        rng = np.random.default_rng(T * 1000 + N)
        V = W.quantize(rng.standard_normal((T, N, d)).astype(np.float32), dtype)
        t = W.quantize(rng.standard_normal(d).astype(np.float32), dtype)
        got = B.metok_segment_score_events(P.to_torch(V, dtype), k, P.to_torch(t, dtype))
        want = O.segment_events(V, k)
        if T > 1:
            P.check_scores(got["sims"].cpu().numpy(), want["sims"], dtype, "sims")
        P.check_scores(got["token_score"].cpu().numpy(), O.token_relevance(V, t), dtype, "token_score")
        assert np.array_equal(got["event_offsets"].cpu().numpy(), want["event_offsets"]) or T <= 3


# ------------------------------------------------------------- a2 a3 a4 ---- #

@pytest.mark.parametrize("name", ["tiny", "frames32", "frames64", "frames128", "frames128d1024"])
def test_compress_vision_workloads(name):
    cfg = W.CONFIGS[name]
    vis = vis_of(name)
    rep = R.compress_case(vis["V"], vis["t"], vis["event_offsets"], cfg.dtype, cfg.alpha, cfg.keep_enc, cfg.keep_enc)
    assert "event_class_flip" not in rep
    assert rep["key_mismatches"] <= rep["key_near_ties"]
    assert rep["assign_mismatches"] <= rep["assign_near_ties"]
    # ceilings from the first green run (0 key-token flips, at most 2 assignment flips per workload):
    # a slide of many decisions inside the near-tie band would still be a regression
    assert rep["key_mismatches"] == 0 and rep["assign_mismatches"] <= MAX_ASSIGN_FLIPS
    print(name, rep)


def test_compress_vision_stress():
    cfg = W.CONFIGS["stress"]
    vis = vis_of("stress")
    rep = R.compress_case(vis["V"], vis["t"], vis["event_offsets"], cfg.dtype, cfg.alpha, cfg.keep_enc, cfg.keep_enc)
    assert "event_class_flip" not in rep
    assert rep["key_mismatches"] == 0 and rep["assign_mismatches"] <= 4 * MAX_ASSIGN_FLIPS   # four times the tokens
    print("stress", rep)


@pytest.mark.parametrize("T,N,d,offs,dtype,kk,kn,agg", [
    (4, 4, 8, [0, 4], "bf16", 0.5, 0.5, 0),
    (6, 9, 72, [0, 1, 2, 6], "f32", 0.3, 0.1, 1),
    (12, 36, 136, [0, 3, 4, 9, 12], "bf16", 0.3, 0.1, 0),
    (10, 25, 264, [0, 5, 10], "bf16", 1.0, 1.0, 0),            # keep everything: identity
    (7, 16, 40, [0, 1, 2, 3, 4, 5, 6, 7], "f32", 0.01, 0.01, 0),   # one key token per event
    (5, 130, 64, [0, 2, 5], "bf16", 0.7, 0.05, 1),
    (14, 64, 72, [0, 12, 14], "bf16", 0.004, 0.004, 0),        # 768 tokens, 4 keys: member lists long enough to be split
    (20, 100, 40, [0, 20], "f32", 0.0005, 0.0005, 0),          # one key token, 1999 members
])
def test_compress_vision_ragged(T, N, d, offs, dtype, kk, kn, agg):
    rng = np.random.default_rng(T * 100 + N)
    base = rng.standard_normal((len(offs) - 1, N, d))
    V = np.concatenate([base[e][None] + 0.3 * rng.standard_normal((offs[e + 1] - offs[e], N, d))
                        for e in range(len(offs) - 1)]).astype(np.float32)
    V = W.quantize(V, dtype)
    t = W.quantize(rng.standard_normal(d).astype(np.float32), dtype)
    rep = R.compress_case(V, t, np.array(offs, dtype=np.int32), dtype, 0.5, kk, kn, agg)
    if kk == 1.0:
        assert rep["n_out"] == T * N


def test_compress_vision_identity_is_bit_exact_and_repeatable():
    cfg = W.CONFIGS["frames32"]
    vis = vis_of("frames32")
    V = P.to_torch(vis["V"][:6], "bf16")
    offs = torch.tensor([0, 2, 6], dtype=torch.int32).cuda()
    t = P.to_torch(vis["t"], "bf16")
    out = B.metok_compress_vision(V, offs, t, B.vision_params(0.5, 1.0, 1.0))
    n = int(out["n_out"].item())
    assert n == 6 * cfg.N
    assert torch.equal(out["out_feats"][:n].view(torch.int16), V.reshape(n, -1).view(torch.int16))
    assert torch.all(out["out_members"][:n] == 1)
    p = B.vision_params(0.5, 0.3, 0.3)
    a = B.metok_compress_vision(V, offs, t, p)
    for _ in range(3):
        b = B.metok_compress_vision(V, offs, t, p)
        m = int(b["n_out"].item())
        assert m == int(a["n_out"].item())
        for key in ("out_feats", "out_src", "out_members"):              # rows beyond n_out are untouched
            x, y = a[key][:m], b[key][:m]
            assert torch.equal(x.view(torch.int16) if x.dtype == torch.bfloat16 else x,
                               y.view(torch.int16) if y.dtype == torch.bfloat16 else y), key
        for key in ("assign", "token_score"):
            assert torch.equal(a[key], b[key]), key


# ------------------------------------------------ Algorithm 1 pooling ------ #

@pytest.mark.parametrize("name", ["tiny", "frames32", "frames64", "frames128d1024", "frames128", "stress"])
def test_compress_vision_pool_workloads(name):
    cfg = W.CONFIGS[name]
    vis = vis_of(name)
    rep = R.pool_case(vis["V"], vis["t"], vis["event_offsets"], cfg.dtype, cfg.alpha, 0.45, (2, 3, 4, 6))
    print(name, rep)
    assert rep["stride_flips"] == 0


@pytest.mark.parametrize("T,G,d,offs,dtype,beta,strides,agg", [
    (5, 3, 8, [0, 2, 5], "bf16", 0.5, (1, 2, 2, 3), 0),
    (9, 5, 72, [0, 1, 4, 9], "f32", 0.3, (2, 3, 4, 5), 1),
    (7, 7, 136, [0, 7], "bf16", 1.0, (3, 3, 7, 8), 0),             # one event; a stride beyond the grid
    (6, 4, 1032, [0, 3, 6], "bf16", 0.01, (1, 1, 1, 1), 0),        # stride 1 everywhere: identity
])
def test_compress_vision_pool_ragged(T, G, d, offs, dtype, beta, strides, agg):
    rng = np.random.default_rng(T * 10 + G)
    N = G * G
    V = W.quantize(rng.standard_normal((T, N, d)).astype(np.float32), dtype)
    t = W.quantize(rng.standard_normal(d).astype(np.float32), dtype)
    rep = R.pool_case(V, t, np.array(offs, dtype=np.int32), dtype, 0.5, beta, strides, agg)
    if strides == (1, 1, 1, 1):
        assert rep["n_out"] == T * N and rep["feature_err"] == 0.0


# ------------------------------------------------------------- a5 a6 a7 ---- #

def _prefill_stage_inputs(cfg, stage, vis):
    """Shapes of the schedule: stage s sees the survivors of stage s-1."""
    grp_full = W.token_groups(cfg, cfg.Nv, vis=vis)
    N0 = [int((grp_full == 0).sum()), int((grp_full == 1).sum())]
    if stage == 1:
        groups = grp_full
    else:
        prev = O.retention_budgets(cfg.alpha, cfg.keep_prefill, stage - 1, N0)
        groups = W.token_groups(cfg, int(prev.sum()), n_key=int(prev[0]), stage=stage)
    budgets = O.retention_budgets(cfg.alpha, cfg.keep_prefill, stage, N0).tolist()
    return groups, budgets


@pytest.mark.parametrize("name,stage", [("tiny", 1), ("frames32", 1), ("frames32", 2), ("frames64", 1),
                                        ("frames64", 2), ("frames64", 3),
                                        ("frames128", 1), ("frames128", 2), ("frames128", 3)])
def test_prefill_prune_workloads(name, stage):
    cfg = W.CONFIGS[name]
    vis = vis_of(name if name != "frames128" else "frames128d1024")
    groups, budgets = _prefill_stage_inputs(cfg, stage, vis)
    n_vis = groups.size
    pf = W.prefill_inputs(cfg, stage, n_vis, groups)
    hidden = W.payload_torch(W.hidden_salt(cfg, stage), pf["S"], cfg.D, cfg.dtype, "cuda")
    rep = R.prefill_case(pf["Q"], pf["K"], cfg.dtype, 0, n_vis, groups, budgets, cfg.dh ** -0.5, hidden)
    assert rep["S_out"] == cfg.Lt + sum(min(b, int((groups == g).sum())) for g, b in enumerate(budgets))
    assert rep["mismatches"] == 0                              # the first green run had none on any workload
    print(name, stage, rep)


@pytest.mark.parametrize("stage", [1, 2, 3])
def test_prefill_prune_stress(stage):
    cfg = W.CONFIGS["stress"]
    vis = vis_of("stress")
    groups, budgets = _prefill_stage_inputs(cfg, stage, vis)
    pf = W.prefill_inputs(cfg, stage, groups.size, groups)
    hidden = W.payload_torch(W.hidden_salt(cfg, stage), pf["S"], cfg.D, cfg.dtype, "cuda")
    rep = R.prefill_case(pf["Q"], pf["K"], cfg.dtype, 0, groups.size, groups, budgets, cfg.dh ** -0.5, hidden)
    assert rep["mismatches"] <= 2
    print("stress", stage, rep)


@pytest.mark.parametrize("Hq,Hkv,Lt,dh,n_vis,vis_start,G,dtype", [
    (1, 1, 1, 64, 5, 0, 1, "f32"), (4, 2, 3, 64, 70, 2, 3, "bf16"), (6, 2, 5, 128, 333, 7, 2, "bf16"),
    (3, 3, 9, 32, 129, 0, 4, "f32"), (8, 1, 17, 128, 1000, 64, 2, "bf16"), (2, 2, 70, 64, 64, 1, 1, "bf16"),
    (2, 1, 4, 64, 2003, 5, 40, "bf16"), (2, 2, 3, 64, 4099, 33, 12, "f32")])
def test_prefill_prune_ragged(Hq, Hkv, Lt, dh, n_vis, vis_start, G, dtype):
    rng = np.random.default_rng(Hq * 100 + n_vis)
    S = vis_start + n_vis + 3 + Lt                              # 3 extra non-visual tokens before the text queries
    Q = W.quantize(rng.standard_normal((Hq, Lt, dh)).astype(np.float32), dtype)
    K = W.quantize(rng.standard_normal((Hkv, S, dh)).astype(np.float32), dtype)
    groups = rng.integers(0, G, size=n_vis).astype(np.int32)
    budgets = [int(rng.integers(0, n_vis // G + 3)) for _ in range(G)]
    budgets[0] = 0 if G > 1 else budgets[0]                     # a class that keeps nothing
    hidden = W.payload_torch(5, S, 24, dtype, "cuda")
    R.prefill_case(Q, K, dtype, vis_start, n_vis, groups, budgets, 0.3, hidden)
    big = [n_vis + 5] * G                                       # budgets above the population keep everything
    rep = R.prefill_case(Q, K, dtype, vis_start, n_vis, groups, big, 0.3, hidden)
    assert rep["S_out"] == S


def test_prefill_prune_tied_scores_keep_lower_index():
    # identical keys => identical scores: the budget must take the lowest indices of each class
    Hq, Lt, dh, n_vis = 2, 2, 64, 50
    Q = np.ones((Hq, Lt, dh), dtype=np.float32)
    K = np.ones((1, n_vis + Lt, dh), dtype=np.float32)
    groups = (np.arange(n_vis) % 2).astype(np.int32)
    got = B.metok_prefill_prune(P.to_torch(Q, "bf16"), P.to_torch(K, "bf16"), None, 0, n_vis,
                                torch.from_numpy(groups).cuda(), [3, 4], 0.125)
    n = int(got["S_out"].item())
    assert got["keep_idx"][:n].cpu().tolist() == [0, 1, 2, 3, 4, 5, 7, 50, 51]


def test_prefill_prune_thousands_of_tied_scores():
    # far more equal scores than one bucket's candidate list holds: the search has to go on
    # over the index part of the keys, and still take the lowest indices of each class
    Hq, Lt, dh, n_vis, vis_start = 2, 2, 64, 5003, 6
    S = vis_start + n_vis + Lt
    Q = np.ones((Hq, Lt, dh), dtype=np.float32)
    K = np.ones((1, S, dh), dtype=np.float32)
    groups = (np.arange(n_vis) % 3).astype(np.int32)
    budgets = [700, 0, 1500]
    got = B.metok_prefill_prune(P.to_torch(Q, "bf16"), P.to_torch(K, "bf16"), None, vis_start, n_vis,
                                torch.from_numpy(groups).cuda(), budgets, 0.125)
    n = int(got["S_out"].item())
    want = list(range(vis_start))
    vis = sorted([vis_start + i for i in range(n_vis) if i % 3 == 0][:700] +
                 [vis_start + i for i in range(n_vis) if i % 3 == 2][:1500])
    want += vis + list(range(vis_start + n_vis, S))
    assert n == len(want)
    assert got["keep_idx"][:n].cpu().tolist() == want
    # two score levels, the cut inside the lower one
    K2 = K.copy()
    K2[0, vis_start:vis_start + 300] *= 2.0
    got = B.metok_prefill_prune(P.to_torch(Q, "bf16"), P.to_torch(K2, "bf16"), None, vis_start, n_vis,
                                torch.zeros(n_vis, dtype=torch.int32).cuda(), [1000], 0.125)
    n = int(got["S_out"].item())
    assert got["keep_idx"][:n].cpu().tolist() == list(range(vis_start + 1000)) + list(range(vis_start + n_vis, S))


# ------------------------------------------------------------- a8 a9 ------- #

@pytest.mark.parametrize("name,policy", [("tiny", O.KV_TOPK), ("tiny", O.KV_PAPER), ("tiny", O.KV_GIVEN),
                                         ("frames32", O.KV_TOPK), ("frames32", O.KV_PAPER),
                                         ("frames32", O.KV_GIVEN), ("frames64", O.KV_TOPK),
                                         ("frames128", O.KV_TOPK), ("frames128", O.KV_PAPER)])
def test_kv_compact_workloads(name, policy):
    cfg = W.CONFIGS[name]
    l1 = 3 if cfg.L > 3 else 0
    rep = R.kv_case(cfg, policy, l1=l1, given_from=7)
    print(name, policy, rep)


@pytest.mark.parametrize("policy", [O.KV_TOPK, O.KV_PAPER, O.KV_GIVEN])
def test_kv_compact_stress(policy):
    rep = R.kv_case(W.CONFIGS["stress"], policy, sample_slabs=4, given_from=11)
    assert rep["slabs_checked"] >= 200
    torch.cuda.empty_cache()


def test_kv_compact_given_lists_are_checked_before_use():
    """Policy GIVEN with lists that would index outside the cache (an entry >= S_cur, a negative
    entry, a descending pair, a repeated entry, a length beyond S_cur): those layers stay bit-identical
    and report S_cur rows, the status word says invalid argument, the good layers are compacted."""
    import dataclasses
    cfg = dataclasses.replace(W.CONFIGS["frames32"], T=6, N=40, L=7, kv_text=9)
    S_cur = cfg.Nv + cfg.kv_text
    ks, vs = W.kv_cache_torch(cfg, torch.device("cuda"), cfg.L)
    before = [(k_.clone(), v_.clone()) for k_, v_ in zip(ks, vs)]
    rng = np.random.default_rng(31)
    good = [np.sort(rng.choice(S_cur, size=n, replace=False)).astype(np.int32) for n in (60, 200)]
    lists = {0: good[0], 1: np.array([3, 9, S_cur, S_cur + 5]), 2: np.array([-4, 2, 7]), 3: np.array([5, 9, 8, 30]),
             4: good[1], 5: np.array([1, 4, 4, 11]), 6: np.arange(S_cur)}
    lens = {l: len(v) for l, v in lists.items()}
    lens[6] = S_cur + 3                                        # longer than the cache
    ki = torch.zeros((cfg.L, S_cur), dtype=torch.int32)
    for l, v in lists.items():
        ki[l, : len(v)] = torch.from_numpy(np.asarray(v, dtype=np.int32))
    got = B.metok_kv_compact(ks, vs, S_cur, O.KV_GIVEN, 0, cfg.Nv, keep_idx=ki.cuda(),
                             keep_len=torch.tensor([lens[l] for l in range(cfg.L)], dtype=torch.int32).cuda())
    torch.cuda.synchronize()
    assert int(got["status"].item()) == -1
    new_len = got["new_len"].cpu().tolist()
    assert new_len == [60, S_cur, S_cur, S_cur, 200, S_cur, S_cur]
    for l in (1, 2, 3, 5, 6):
        assert torch.equal(ks[l].view(torch.int16), before[l][0].view(torch.int16))
        assert torch.equal(vs[l].view(torch.int16), before[l][1].view(torch.int16))
    for l, lst in ((0, good[0]), (4, good[1])):
        idx = torch.from_numpy(lst.astype(np.int64)).cuda()
        assert torch.equal(ks[l][:, : len(lst)].view(torch.int16), before[l][0][:, idx].view(torch.int16))
        assert torch.equal(vs[l][:, : len(lst)].view(torch.int16), before[l][1][:, idx].view(torch.int16))
    # all lists good: status OK
    ks2, vs2 = W.kv_cache_torch(cfg, torch.device("cuda"), 2)
    ki2 = torch.zeros((2, S_cur), dtype=torch.int32)
    for l in range(2):
        ki2[l, : len(good[l])] = torch.from_numpy(good[l])
    ok = B.metok_kv_compact(ks2, vs2, S_cur, O.KV_GIVEN, 0, cfg.Nv, keep_idx=ki2.cuda(),
                            keep_len=torch.tensor([60, 200], dtype=torch.int32).cuda())
    torch.cuda.synchronize()
    assert int(ok["status"].item()) == 0 and ok["new_len"].cpu().tolist() == [60, 200]


def test_kv_compact_per_layer_scores():
    R.kv_case(W.CONFIGS["frames32"], O.KV_TOPK, per_layer_scores=True)


@pytest.mark.parametrize("ratio", [0.0, 0.03, 0.5, 0.97, 1.0])
def test_kv_compact_ratios_and_fp32_rows(ratio):
    import dataclasses
    cfg = dataclasses.replace(W.CONFIGS["tiny"], T=37, N=29, dh=36, Hkv=3, L=5, kv_text=11, keep_kv=ratio)
    R.kv_case(cfg, O.KV_TOPK)
    cfg2 = dataclasses.replace(W.CONFIGS["frames32"], T=9, N=33, dh=24, Hkv=2, L=3, kv_text=5, keep_kv=ratio)
    R.kv_case(cfg2, O.KV_TOPK)


# ------------------------------------------------------------- chained ----- #

def test_chained_pipeline_tiny_and_frames32():
    """segment -> compress on the GPU's own event offsets; both must equal the oracle's chain."""
    for name in ("tiny", "frames32"):
        cfg = W.CONFIGS[name]
        vis = vis_of(name)
        Vd = P.to_torch(vis["V"], cfg.dtype)
        seg = B.metok_segment_events(Vd, cfg.k)
        p = B.vision_params(cfg.alpha, cfg.keep_enc, cfg.keep_enc)
        out = B.metok_compress_vision(Vd, seg["event_offsets"], P.to_torch(vis["t"], cfg.dtype), p)
        want_seg = O.segment_events(vis["V"], cfg.k)
        want = O.compress_vision(vis["V"], vis["t"], want_seg["event_offsets"], cfg.alpha, cfg.keep_enc,
                                 cfg.keep_enc, cfg.dtype)
        n = int(out["n_out"].item())
        assert n == want["n_out"]
        assert np.array_equal(out["event_is_key"].cpu().numpy(), want["event_is_key"])
        same = np.mean(out["out_src"][:n].cpu().numpy() == want["out_src"])
        assert same > 0.99


# ---------------------------------------- other model sizes, ablation settings ----- #

@pytest.mark.parametrize("name,l1", [("small24", 3), ("large40", 13)])
def test_other_model_sizes_all_four_calls(name, l1):
    """The paper's smallest and largest decoders (24 layers, 14/2 heads of 64; 40 layers, 40 heads of
    128 without head sharing): every call at those shapes, three pruning levels, both K/V policies."""
    cfg = W.CONFIGS[name]
    vis = vis_of(name)
    Vd, td = P.to_torch(vis["V"], cfg.dtype), P.to_torch(vis["t"], cfg.dtype)
    got = B.metok_segment_score_events(Vd, cfg.k, td)
    want = O.segment_events(vis["V"], cfg.k)
    P.check_scores(got["sims"].cpu().numpy(), want["sims"], cfg.dtype, "sims")
    assert np.array_equal(got["event_offsets"].cpu().numpy(), want["event_offsets"])
    assert np.array_equal(want["event_offsets"], vis["event_offsets"])
    rep = R.compress_case(vis["V"], vis["t"], vis["event_offsets"], cfg.dtype, cfg.alpha, cfg.keep_enc, cfg.keep_enc)
    assert "event_class_flip" not in rep
    assert rep["key_mismatches"] <= rep["key_near_ties"] and rep["assign_mismatches"] <= rep["assign_near_ties"]
    for stage in (1, 2, 3):
        groups, budgets = _prefill_stage_inputs(cfg, stage, vis)
        pf = W.prefill_inputs(cfg, stage, groups.size, groups)
        hidden = W.payload_torch(W.hidden_salt(cfg, stage), pf["S"], cfg.D, cfg.dtype, "cuda")
        r = R.prefill_case(pf["Q"], pf["K"], cfg.dtype, 0, groups.size, groups, budgets, cfg.dh ** -0.5, hidden)
        assert r["S_out"] == cfg.Lt + sum(min(b, int((groups == g).sum())) for g, b in enumerate(budgets))
    del hidden
    torch.cuda.empty_cache()
    R.kv_case(cfg, O.KV_TOPK)
    R.kv_case(cfg, O.KV_PAPER, l1=l1)


def test_ablation_uniform_segmentation_max_events_last_token_scores():
    """Settings of the paper's ablations that are arguments of the calls: events of equal length
    instead of Eq. 4's (the caller's offsets), the event score as the maximum over frames
    (Algorithm 1), and attention scores from the last text token alone (one query row)."""
    cfg = W.CONFIGS["frames32"]
    vis = vis_of("frames32")
    uniform = np.linspace(0, cfg.T, cfg.k + 1).round().astype(np.int32)
    assert not np.array_equal(uniform, vis["event_offsets"])
    for agg in (O.AGG_MEAN, O.AGG_MAX):
        rep = R.compress_case(vis["V"], vis["t"], uniform, cfg.dtype, cfg.alpha, cfg.keep_enc, cfg.keep_enc, agg)
        assert "event_class_flip" not in rep
        assert rep["key_mismatches"] <= rep["key_near_ties"] and rep["assign_mismatches"] <= rep["assign_near_ties"]
    groups, budgets = _prefill_stage_inputs(cfg, 1, vis)
    pf = W.prefill_inputs(cfg, 1, cfg.Nv, groups)
    # the keys of the earlier text tokens stay in the sequence; only the last one asks
    r = R.prefill_case(pf["Q"][:, -1:, :], pf["K"], cfg.dtype, 0, cfg.Nv, groups, budgets, cfg.dh ** -0.5)
    assert r["S_out"] == cfg.Lt + sum(min(b, int((groups == g).sum())) for g, b in enumerate(budgets))


def test_cuda_graph_replay_equals_eager_calls():
    """The four calls enqueue on a stream and never synchronise: captured once in a CUDA graph
    (kernel-to-kernel edges become programmatic ones) and replayed, they must leave exactly what
    the eager calls leave."""
    cfg = W.CONFIGS["frames32"]
    vis = vis_of("frames32")
    Vd, td = P.to_torch(vis["V"], cfg.dtype), P.to_torch(vis["t"], cfg.dtype)
    p = B.vision_params(cfg.alpha, cfg.keep_enc, cfg.keep_enc)
    groups, budgets = _prefill_stage_inputs(cfg, 1, vis)
    pf = W.prefill_inputs(cfg, 1, cfg.Nv, groups)
    Q, K = P.to_torch(pf["Q"], cfg.dtype), P.to_torch(pf["K"], cfg.dtype)
    hidden = W.payload_torch(W.hidden_salt(cfg, 1), pf["S"], cfg.D, cfg.dtype, "cuda")
    grp = torch.from_numpy(groups.astype(np.int32)).cuda()
    S_cur = cfg.Nv + cfg.kv_text
    layers = 4

    def step(o, ks, vs):
        o["seg"] = B.metok_segment_score_events(Vd, cfg.k, td, out=o.get("seg"))
        o["cv"] = B.metok_compress_vision(Vd, o["seg"]["event_offsets"], td, p, out=o.get("cv"), scored=o["seg"])
        o["pf"] = B.metok_prefill_prune(Q, K, hidden, 0, cfg.Nv, grp, budgets, cfg.dh ** -0.5, out=o.get("pf"))
        kv = o.get("kv") or {"keep_idx": None, "keep_len": None, "new_len": None}
        o["kv"] = B.metok_kv_compact(ks, vs, S_cur, B.KV_TOPK, 0, cfg.Nv, keep_ratio=cfg.keep_kv,
                                     scores=o["pf"]["scores"], keep_idx=kv["keep_idx"], keep_len=kv["keep_len"],
                                     new_len=kv["new_len"])

    def caches():
        return W.kv_cache_torch(cfg, torch.device("cuda"), layers)

    side = torch.cuda.Stream()
    eager, replay = {}, {}
    ks_e, vs_e = caches()
    ks_g, vs_g = caches()
    with torch.cuda.stream(side):
        step(eager, ks_e, vs_e)
        scratch_k, scratch_v = caches()
        step(replay, scratch_k, scratch_v)                     # allocates the outputs the graph will write
    side.synchronize()
    for d in replay.values():                                   # nothing of the warm-up may survive by accident
        for t in d.values():
            if isinstance(t, torch.Tensor) and t.numel() and not t.dtype.is_floating_point:
                t.fill_(-1) if t.dtype != torch.uint8 else t.fill_(255)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step(replay, ks_g, vs_g)
    graph.replay()
    torch.cuda.synchronize()

    def same(a, b):
        return torch.equal(a.view(torch.int16) if a.dtype == torch.bfloat16 else a,
                           b.view(torch.int16) if b.dtype == torch.bfloat16 else b)

    for name in ("sims", "boundaries", "event_offsets", "frame_event", "token_score", "token_inv_norm"):
        assert same(eager["seg"][name], replay["seg"][name]), name
    n = int(eager["cv"]["n_out"].item())
    assert n == int(replay["cv"]["n_out"].item()) and n > 0
    for name in ("out_feats", "out_src", "out_event", "out_members"):
        assert same(eager["cv"][name][:n], replay["cv"][name][:n]), name
    for name in ("assign", "frame_score", "event_score", "event_is_key"):
        assert same(eager["cv"][name], replay["cv"][name]), name
    s_out = int(eager["pf"]["S_out"].item())
    assert s_out == int(replay["pf"]["S_out"].item())
    assert same(eager["pf"]["scores"], replay["pf"]["scores"])
    assert same(eager["pf"]["keep_idx"][:s_out], replay["pf"]["keep_idx"][:s_out])
    assert same(eager["pf"]["hidden_out"][:s_out], replay["pf"]["hidden_out"][:s_out])
    new_len = eager["kv"]["new_len"].cpu().tolist()
    assert new_len == replay["kv"]["new_len"].cpu().tolist()
    for layer in range(layers):
        m = new_len[layer]
        assert same(eager["kv"]["keep_idx"][layer, :m], replay["kv"]["keep_idx"][layer, :m])
        assert same(ks_e[layer][:, :m], ks_g[layer][:, :m]) and same(vs_e[layer][:, :m], vs_g[layer][:, :m])


@pytest.mark.parametrize("name", ["frames32", "small24", "tiny", "frames128"])
def test_prefill_prune_schedule_three_levels_in_one_call(name):
    """The pruning levels chained on the device (classes and origins of the survivors handed from
    level to level without a read-back) against the oracle's chain."""
    cfg = W.CONFIGS[name]
    vis = vis_of(name if name != "frames128" else "frames128d1024")   # only the events' classes are used
    groups = W.token_groups(cfg, cfg.Nv, vis=vis)
    N0 = [int((groups == 0).sum()), int((groups == 1).sum())]
    n_levels = 3 if N0[0] > 3 else 2
    r = cfg.keep_prefill
    sizes = B.metok_prune_schedule_sizes(n_levels, cfg.alpha, r, N0)
    # inputs of level s depend on who survived level s-1: generated along the oracle's chain
    Qs, Ks, hid = [], [], []
    g_s = groups
    for s in range(1, n_levels + 1):
        assert g_s.size == sizes[s - 1]
        pf = W.prefill_inputs(cfg, s, g_s.size, g_s)
        Qs.append(pf["Q"]); Ks.append(pf["K"])
        hid.append(W.payload_torch(W.hidden_salt(cfg, s), pf["S"], cfg.D, cfg.dtype, "cuda"))
        want_s = O.prune_schedule(Qs, Ks, groups, cfg.alpha, r, 0, O.f32(cfg.dh ** -0.5))
        k_ = want_s[-1]["keep_idx"]
        g_s = g_s[k_[k_ < g_s.size]]
    want = want_s
    got = B.metok_prefill_prune_schedule([P.to_torch(q, cfg.dtype) for q in Qs], [P.to_torch(k_, cfg.dtype) for k_ in Ks],
                                         hid, 0, torch.from_numpy(groups.astype(np.int32)).cuda(), cfg.alpha, r, N0,
                                         cfg.dh ** -0.5)
    torch.cuda.synchronize()
    assert int(got[0]["status"].item()) == 0
    for s in range(n_levels):
        w, g = want[s], got[s]
        n_in = sizes[s]
        assert g["n_vis"] == n_in == w["token_group"].size
        assert np.array_equal(g["token_group"][:n_in].cpu().numpy(), w["token_group"]), s
        assert np.array_equal(g["origin"][:n_in].cpu().numpy(), w["origin"]), s
        P.check_scores(g["scores"][:n_in].cpu().numpy(), w["scores"], cfg.dtype, f"scores of level {s + 1}")
        S_out = int(g["S_out"].item())
        assert S_out == w["S_out"] == g["S"] - n_in + sizes[s + 1]
        keep = g["keep_idx"][:S_out].cpu().numpy()
        mism = P.check_index_set(keep, w["keep_idx"], lambda u: u < n_in and bool(w["near_tie"][u]), "keep_idx")
        ho = g["hidden_out"][:S_out]
        ref = hid[s][torch.from_numpy(keep.astype(np.int64)).cuda()]
        assert torch.equal(ho.view(torch.int16) if ho.dtype == torch.bfloat16 else ho,
                           ref.view(torch.int16) if ref.dtype == torch.bfloat16 else ref)
        if mism:                                               # a near-tie went the other way: later levels see other tokens
            break
    # wrong class counts are reported by the device status word
    bad = [N0[0] + 1, N0[1] - 1]
    if bad[1] >= 0 and min(B.metok_prune_schedule_sizes(n_levels, cfg.alpha, r, bad)[:n_levels]) > 0:
        sz = B.metok_prune_schedule_sizes(n_levels, cfg.alpha, r, bad)
        Ks_bad = [torch.zeros((cfg.Hkv, Ks[0].shape[1] - cfg.Nv + sz[s], cfg.dh), dtype=P.to_torch(Ks[0], cfg.dtype).dtype,
                              device="cuda") for s in range(n_levels)]
        out = B.metok_prefill_prune_schedule([P.to_torch(q, cfg.dtype) for q in Qs], Ks_bad, None, 0,
                                             torch.from_numpy(groups.astype(np.int32)).cuda(), cfg.alpha, r, bad,
                                             cfg.dh ** -0.5)
        torch.cuda.synchronize()
        assert int(out[0]["status"].item()) == -1


def test_kv_lists_from_the_recorded_keep_lists_and_their_compaction():
    """The schedule's recorded keep lists as K/V lists per layer (metok_prune_schedule_kv_lists), equal to
    the oracle's, and the caches of every layer group compacted with them (policy GIVEN) equal to the
    oracle's gather."""
    import dataclasses
    cfg = dataclasses.replace(W.CONFIGS["frames32"], L=6)
    vis = vis_of("frames32")
    groups = W.token_groups(cfg, cfg.Nv, vis=vis)
    N0 = [int((groups == 0).sum()), int((groups == 1).sum())]
    r, layers = cfg.keep_prefill, [1, 3, 4]
    sizes = B.metok_prune_schedule_sizes(3, cfg.alpha, r, N0)
    Qs, Ks, g_s = [], [], groups
    for s in range(1, 4):
        pf = W.prefill_inputs(cfg, s, g_s.size, g_s)
        Qs.append(pf["Q"]); Ks.append(pf["K"])
        want_lv = O.prune_schedule(Qs, Ks, groups, cfg.alpha, r, 0, O.f32(cfg.dh ** -0.5))
        k_ = want_lv[-1]["keep_idx"]
        g_s = g_s[k_[k_ < g_s.size]]
    S = cfg.Nv + cfg.Lt
    got_lv = B.metok_prefill_prune_schedule([P.to_torch(q, cfg.dtype) for q in Qs], [P.to_torch(k_, cfg.dtype) for k_ in Ks],
                                            None, 0, torch.from_numpy(groups.astype(np.int32)).cuda(), cfg.alpha, r, N0,
                                            cfg.dh ** -0.5)
    kv = B.metok_prune_schedule_kv_lists(got_lv, layers, cfg.L)
    torch.cuda.synchronize()
    want = O.schedule_kv_lists(want_lv, layers, cfg.L, S)
    lens = kv["keep_len"].cpu().numpy()
    same_lists = all(np.array_equal(got_lv[s]["keep_idx"][: int(got_lv[s]["S_out"].item())].cpu().numpy(), want_lv[s]["keep_idx"])
                     for s in range(3))
    for l in range(cfg.L):
        grp = sum(1 for x in layers if x <= l)
        assert kv["S_cur"][l] == S - cfg.Nv + sizes[grp]
        assert lens[l] == want[l].size
        if same_lists:                                       # (a near-tie may tip a level's list; the sizes hold either way)
            assert np.array_equal(kv["keep_idx"][l, : lens[l]].cpu().numpy(), want[l]), l
    # compaction per layer group with the lists as given ones
    for grp_layers in ([0], [1, 2], [3], [4, 5]):
        S_cur = kv["S_cur"][grp_layers[0]]
        ks = [W.payload_torch(900 + l, cfg.Hkv * S_cur, cfg.dh, cfg.dtype, "cuda").view(cfg.Hkv, S_cur, cfg.dh) for l in grp_layers]
        vs = [W.payload_torch(950 + l, cfg.Hkv * S_cur, cfg.dh, cfg.dtype, "cuda").view(cfg.Hkv, S_cur, cfg.dh) for l in grp_layers]
        before = [(a.clone(), b.clone()) for a, b in zip(ks, vs)]
        ki = torch.zeros((len(grp_layers), S_cur), dtype=torch.int32, device="cuda")
        for j, l in enumerate(grp_layers):
            ki[j, : lens[l]] = kv["keep_idx"][l, : lens[l]]
        out = B.metok_kv_compact(ks, vs, S_cur, O.KV_GIVEN, 0, S_cur - cfg.Lt, keep_idx=ki,
                                 keep_len=kv["keep_len"][grp_layers[0]: grp_layers[-1] + 1].clone())
        torch.cuda.synchronize()
        assert int(out["status"].item()) == 0
        for j, l in enumerate(grp_layers):
            idx = kv["keep_idx"][l, : lens[l]].long()
            assert torch.equal(ks[j][:, : lens[l]].view(torch.int16), before[j][0][:, idx].view(torch.int16))
            assert torch.equal(vs[j][:, : lens[l]].view(torch.int16), before[j][1][:, idx].view(torch.int16))


def test_two_videos_on_two_streams_do_not_share_scratch():
    """Independent videos in flight on streams of their own (the benchmark's batch): each call takes
    its scratch per stream, so the results equal those of the same calls made one after the other."""
    cfg = W.CONFIGS["frames32"]
    vis = vis_of("frames32")
    p = B.vision_params(cfg.alpha, cfg.keep_enc, cfg.keep_enc)
    rng = np.random.default_rng(5)
    Va = vis["V"]
    Vb = W.quantize((Va[::-1] + 0.05 * rng.standard_normal(Va.shape)).astype(np.float32), cfg.dtype)
    td = P.to_torch(vis["t"], cfg.dtype)
    vids = [P.to_torch(Va, cfg.dtype), P.to_torch(Vb, cfg.dtype)]

    def one(V):
        seg = B.metok_segment_score_events(V, cfg.k, td)
        cv = B.metok_compress_vision(V, seg["event_offsets"], td, p, scored=seg)
        return seg, cv

    alone = []
    for V in vids:
        alone.append(one(V))
        torch.cuda.synchronize()
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    for _ in range(3):
        both = []
        for V, st in zip(vids, streams):
            with torch.cuda.stream(st):
                both.append(one(V))
        torch.cuda.synchronize()
        for (seg_a, cv_a), (seg_b, cv_b) in zip(alone, both):
            assert torch.equal(seg_a["event_offsets"], seg_b["event_offsets"])
            assert torch.equal(seg_a["token_score"], seg_b["token_score"])
            n = int(cv_a["n_out"].item())
            assert n == int(cv_b["n_out"].item())
            assert torch.equal(cv_a["out_src"][:n], cv_b["out_src"][:n])
            assert torch.equal(cv_a["assign"], cv_b["assign"])
            assert torch.equal(cv_a["out_feats"][:n].view(torch.int16), cv_b["out_feats"][:n].view(torch.int16))
    assert not torch.equal(alone[0][1]["assign"], alone[1][1]["assign"])      # the two videos do differ


@pytest.mark.parametrize("name,world", [("frames32", 2), ("frames32", 4), ("tiny", 1), ("small24", 2)])
def test_head_sharded_scores_then_selection(name, world):
    """The two halves of the pruning call on their own: the scores of each shard of KV-head groups
    (normalised by all heads' rows) add up to the unsharded scores, and the selection on the sum is
    the fused call's.  The shards run one after the other on this GPU; a sum on the device stands in
    for the all-reduce between ranks."""
    cfg = W.CONFIGS[name]
    vis = vis_of(name)
    groups, budgets = _prefill_stage_inputs(cfg, 1, vis)
    pf = W.prefill_inputs(cfg, 1, cfg.Nv, groups)
    Q, K = P.to_torch(pf["Q"], cfg.dtype), P.to_torch(pf["K"], cfg.dtype)
    hidden = W.payload_torch(W.hidden_salt(cfg, 1), pf["S"], cfg.D, cfg.dtype, "cuda")
    grp = torch.from_numpy(groups.astype(np.int32)).cuda()
    scale = cfg.dh ** -0.5
    fused = B.metok_prefill_prune(Q, K, hidden, 0, cfg.Nv, grp, budgets, scale)
    total = torch.zeros(cfg.Nv, dtype=torch.float32, device="cuda")
    for rank in range(world):
        (h0, h1), (g0, g1) = B.head_shard(cfg.Hq, cfg.Hkv, rank, world)
        part = B.metok_attention_scores(Q[h0:h1].contiguous(), K[g0:g1].contiguous(), 0, cfg.Nv, scale,
                                        rows_total=cfg.Hq * cfg.Lt)
        total += part
    torch.cuda.synchronize()
    want_scores = O.attention_scores(pf["Q"], pf["K"], 0, cfg.Nv, O.f32(scale))
    P.check_scores(total.cpu().numpy(), want_scores, cfg.dtype, "sum of the shards' scores")
    assert torch.allclose(total, fused["scores"], rtol=2e-5, atol=1e-9)
    if world == 1:
        assert torch.equal(total, fused["scores"])
    got = B.metok_prune_by_scores(fused["scores"].clone(), hidden, pf["S"], 0, grp, budgets)
    torch.cuda.synchronize()
    n = int(fused["S_out"].item())
    assert int(got["S_out"].item()) == n and int(got["status"].item()) == 0
    assert torch.equal(got["keep_idx"][:n], fused["keep_idx"][:n])
    assert torch.equal(got["hidden_out"][:n].view(torch.int16) if cfg.dtype == "bf16" else got["hidden_out"][:n],
                       fused["hidden_out"][:n].view(torch.int16) if cfg.dtype == "bf16" else fused["hidden_out"][:n])
    # selection on the summed scores against the oracle's selection (near-ties aside)
    sel = B.metok_prune_by_scores(total, None, pf["S"], 0, grp, budgets)
    want = O.weighted_topk(want_scores, groups, budgets, pf["S"], 0)
    m = int(sel["S_out"].item())
    assert m == want["S_out"]
    P.check_index_set(sel["keep_idx"][:m].cpu().numpy(), want["keep_idx"],
                      lambda u: u < cfg.Nv and bool(want["near_tie"][u]), "keep_idx from summed scores")


@pytest.mark.parametrize("name", ["frames32", "frames128"])
def test_head_sharded_call_at_world_size_one_equals_the_fused_call(name):
    """binding.metok_prefill_prune_sharded itself (the function that joins the two halves around the
    all-reduce), run as the only rank: same scores, keep list and hidden rows as metok_prefill_prune,
    bit for bit."""
    cfg = W.CONFIGS[name]
    vis = vis_of(name if name != "frames128" else "frames128d1024")
    groups, budgets = _prefill_stage_inputs(cfg, 1, vis)
    pf = W.prefill_inputs(cfg, 1, cfg.Nv, groups)
    Q, K = P.to_torch(pf["Q"], cfg.dtype), P.to_torch(pf["K"], cfg.dtype)
    hidden = W.payload_torch(W.hidden_salt(cfg, 1), pf["S"], cfg.D, cfg.dtype, "cuda")
    grp = torch.from_numpy(groups.astype(np.int32)).cuda()
    scale = cfg.dh ** -0.5
    fused = B.metok_prefill_prune(Q, K, hidden, 0, cfg.Nv, grp, budgets, scale)
    (h0, h1), (g0, g1) = B.head_shard(cfg.Hq, cfg.Hkv, 0, 1)
    assert (h0, h1, g0, g1) == (0, cfg.Hq, 0, cfg.Hkv)
    got = B.metok_prefill_prune_sharded(Q[h0:h1], K[g0:g1], hidden, 0, cfg.Nv, grp, budgets, scale)
    torch.cuda.synchronize()
    n = int(fused["S_out"].item())
    assert int(got["S_out"].item()) == n and int(got["status"].item()) == 0
    assert torch.equal(got["keep_idx"][:n], fused["keep_idx"][:n])
    assert torch.equal(got["hidden_out"][:n].view(torch.int16), fused["hidden_out"][:n].view(torch.int16))
    want = O.weighted_topk(O.attention_scores(pf["Q"], pf["K"], 0, cfg.Nv, O.f32(scale)), groups, budgets, pf["S"], 0)
    assert n == want["S_out"]
    P.check_index_set(got["keep_idx"][:n].cpu().numpy(), want["keep_idx"],
                      lambda u: u < cfg.Nv and bool(want["near_tie"][u]), "keep_idx of the sharded call")


def test_ablation_key_frames_given_by_the_caller():
    """Randomly chosen key frames (the ablation of Algorithm 1's key-frame choice): the caller's mask
    decides the strides; with a given mask no score can tip a frame, so the layout must match exactly."""
    cfg = W.CONFIGS["frames32"]
    vis = vis_of("frames32")
    rng = np.random.default_rng(41)
    given = (rng.random(cfg.T) < 0.4).astype(np.uint8)
    rep = R.pool_case(vis["V"], vis["t"], vis["event_offsets"], cfg.dtype, cfg.alpha, 0.45, (2, 3, 4, 6), key_frames=given)
    assert rep["stride_flips"] == 0 and rep["n_out"] > 0
    base = R.pool_case(vis["V"], vis["t"], vis["event_offsets"], cfg.dtype, cfg.alpha, 0.45, (2, 3, 4, 6))
    assert rep["n_out"] != base["n_out"]                      # the mask does change the layout


def test_ablation_key_events_given_by_the_caller():
    """Randomly chosen key events (the paper's Table 4 ablation) as an argument: the per-event
    ratios follow the caller's mask, everything else as usual."""
    cfg = W.CONFIGS["frames32"]
    vis = vis_of("frames32")
    rng = np.random.default_rng(17)
    for mask in (rng.random(cfg.k) < 0.5, np.zeros(cfg.k, dtype=bool), np.ones(cfg.k, dtype=bool)):
        rep = R.compress_case(vis["V"], vis["t"], vis["event_offsets"], cfg.dtype, cfg.alpha, 0.3, 0.05,
                              key_events=mask)
        assert "event_class_flip" not in rep
        assert rep["key_mismatches"] <= rep["key_near_ties"] and rep["assign_mismatches"] <= rep["assign_near_ties"]
        want_n = sum(max(1, math.ceil((0.3 if mask[e] else 0.05) * (vis["event_offsets"][e + 1] - vis["event_offsets"][e])
                                      * cfg.N - 1e-9)) for e in range(cfg.k))
        assert rep["n_out"] == want_n


def test_benchmark_launch_configuration_equals_eager_calls_at_full_size():
    """The configuration the benchmark times -- the 128-frame workload, two videos in flight on
    streams of their own, K/V compaction on a side stream, all captured in one CUDA graph -- leaves
    bit for bit what the same calls leave when made eagerly one after the other (those are the calls
    the parity tests above compare with the oracle at this size)."""
    import os
    import sys
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    import bench
    _vis_cache.clear()
    torch.cuda.empty_cache()
    cfg = W.CONFIGS["frames128"]
    dev = torch.device("cuda", 0)
    ref = bench.Workload(cfg, dev, host_copies=False)
    lanes_w = [ref.twin(), ref.twin()]
    ref.step(); ref.step()                                      # two eager passes (the K/V cache is compacted twice)
    for w in lanes_w:
        w.step()                                                # first pass eagerly: allocates the outputs
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream() for _ in lanes_w]
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        main = torch.cuda.current_stream()
        for st in streams:
            st.wait_stream(main)
        for w, st in zip(lanes_w, streams):
            with torch.cuda.stream(st):
                w.step()
        for st in streams:
            main.wait_stream(st)
    graph.replay()                                              # second pass of both videos, concurrently
    torch.cuda.synchronize()

    def same(a, b):
        a = a.view(torch.int16) if a.dtype == torch.bfloat16 else a
        b = b.view(torch.int16) if b.dtype == torch.bfloat16 else b
        return torch.equal(a, b)

    for w in lanes_w:
        o, r = w.out, ref.out
        for name in ("sims", "boundaries", "event_offsets", "frame_event", "token_score"):
            assert same(o["seg"][name], r["seg"][name]), name
        n = int(r["cv"]["n_out"].item())
        assert int(o["cv"]["n_out"].item()) == n
        for name in ("out_feats", "out_src", "out_event", "out_members"):
            assert same(o["cv"][name][:n], r["cv"][name][:n]), name
        assert same(o["cv"]["assign"], r["cv"]["assign"])
        for i in range(len(ref.stages)):
            a, b = o[f"pf{i}"], r[f"pf{i}"]
            s = int(b["S_out"].item())
            assert int(a["S_out"].item()) == s and int(a["status"].item()) == 0
            assert same(a["scores"], b["scores"]) and same(a["keep_idx"][:s], b["keep_idx"][:s])
            assert same(a["hidden_out"][:s], b["hidden_out"][:s])
        nl = r["kv"]["new_len"].cpu().tolist()
        assert o["kv"]["new_len"].cpu().tolist() == nl
        for layer in (0, cfg.L // 2, cfg.L - 1):
            m = nl[layer]
            assert same(o["kv"]["keep_idx"][layer, :m], r["kv"]["keep_idx"][layer, :m])
            assert same(w.ks[layer][:, :m], ref.ks[layer][:, :m]) and same(w.vs[layer][:, :m], ref.vs[layer][:, :m])
    del graph, lanes_w, ref
    torch.cuda.empty_cache()


# ------------------------------------------------- random shapes, all calls ---- #

@pytest.mark.parametrize("seed", list(range(32)))
def test_random_shapes_through_all_calls(seed):
    """Seeded random small shapes, ratios, modes and types through segmentation, both compressors and
    the pruning call: shapes nobody picked by hand (odd head counts, row lengths on and off the
    tensor-core paths, classes without members, budgets of zero and above the population)."""
    rng = np.random.default_rng(9000 + seed)
    dtype = "bf16" if rng.random() < 0.6 else "f32"
    T = int(rng.integers(1, 33))
    Gs = int(rng.integers(1, 9))
    N = Gs * Gs
    d = int(rng.integers(1, 40)) * 8
    k = int(rng.integers(1, T + 1))
    cuts = np.sort(rng.choice(np.arange(1, T), size=k - 1, replace=False)) if k > 1 else np.zeros(0, np.int64)
    offs = np.concatenate([[0], cuts, [T]]).astype(np.int32)
    base = rng.standard_normal((k, N, d))
    V = np.concatenate([base[e][None] + 0.4 * rng.standard_normal((offs[e + 1] - offs[e], N, d)) for e in range(k)])
    V = W.quantize(V.astype(np.float32), dtype)
    t = W.quantize(rng.standard_normal(d).astype(np.float32), dtype)
    for mode in (O.SIM_FLATTEN, O.SIM_MEANPOOL):
        R.segment_case(V, dtype, k, mode)
    alpha = float(rng.choice([0.25, 0.5, 0.75, 1.0]))
    kk, kn = float(rng.choice([0.02, 0.1, 0.3, 0.6, 1.0])), float(rng.choice([0.01, 0.05, 0.2, 0.5]))
    agg = int(rng.integers(0, 2))
    R.compress_case(V, t, offs, dtype, alpha, kk, kn, agg)
    strides = tuple(int(x) for x in rng.integers(1, Gs + 2, size=4))
    R.pool_case(V, t, offs, dtype, alpha, float(rng.choice([0.2, 0.5, 1.0])), strides, agg)

    Hkv = int(rng.integers(1, 4))
    Hq = Hkv * int(rng.integers(1, 5))
    Lt = int(rng.integers(1, 40))
    dh = int(rng.choice([64, 128])) if dtype == "bf16" else int(rng.choice([20, 32, 64, 128]))   # bf16 heads: 64 or 128 only
    n_vis = int(rng.integers(1, 3000))
    vis_start = int(rng.integers(0, 20))
    G = int(rng.integers(1, 6))
    S = vis_start + n_vis + int(rng.integers(0, 4)) + Lt
    Q = W.quantize(rng.standard_normal((Hq, Lt, dh)).astype(np.float32), dtype)
    K = W.quantize(rng.standard_normal((Hkv, S, dh)).astype(np.float32), dtype)
    groups = rng.integers(0, G + 1, size=n_vis).astype(np.int32)
    groups[groups == G] = int(rng.integers(0, G))               # some class may end up without members
    budgets = [int(rng.integers(0, n_vis // G + 3)) for _ in range(G)]
    hidden = W.payload_torch(7 + seed, S, 8 * int(rng.integers(1, 20)), dtype, "cuda")
    R.prefill_case(Q, K, dtype, vis_start, n_vis, groups, budgets, float(dh) ** -0.5, hidden)


@pytest.mark.parametrize("seed", list(range(16)))
def test_random_kv_caches(seed):
    """Seeded random cache shapes, ratios and policies through the K/V selection and in-place gather."""
    import dataclasses
    rng = np.random.default_rng(7000 + seed)
    cfg = dataclasses.replace(
        W.CONFIGS["tiny"], name=f"rand{seed}", index=100 + seed, T=int(rng.integers(1, 40)), N=int(rng.integers(1, 60)),
        dtype="bf16" if rng.random() < 0.6 else "f32", Hkv=int(rng.integers(1, 5)),
        dh=int(rng.choice([8, 32, 64, 128])), L=int(rng.integers(1, 7)),
        keep_kv=float(rng.choice([0.0, 0.01, 0.065, 0.3, 0.8, 1.0])), kv_text=int(rng.integers(0, 30)))
    policy = [O.KV_TOPK, O.KV_PAPER, O.KV_GIVEN][seed % 3]
    R.kv_case(cfg, policy, per_layer_scores=bool(seed & 4), l1=int(rng.integers(0, cfg.L + 1)), sample_slabs=4,
              given_from=seed)

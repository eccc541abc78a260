"""Run one C-ABI call on the GPU and the oracle on the CPU from the same seeded
inputs, compare under the parity protocol (tests/parity.py), return a report.
Shared by the parity tests and by the smoke check."""

from __future__ import annotations

from typing import Dict, Optional, Sequence

import numpy as np
import torch

from oracle import metok_oracle as O
from paper_2506_02850_b200 import binding as B
from paper_2506_02850_b200 import workloads as W

from . import parity as P


def segment_case(V: np.ndarray, dtype: str, k: int, sim_mode: int = 0) -> Dict[str, object]:
    want = O.segment_events(V, k, sim_mode)
    got = B.metok_segment_events(P.to_torch(V, dtype), k, sim_mode)
    torch.cuda.synchronize()
    T = V.shape[0]
    rep = {"near_ties": 0, "mismatches": 0}
    if T > 1:
        rep["sims_err"] = P.check_scores(got["sims"].cpu().numpy(), want["sims"], dtype, "sims")
    gb, wb = got["boundaries"].cpu().numpy(), want["boundaries"]
    if not np.array_equal(gb, wb):
        # only excusable when the (k-1)-th and k-th smallest similarities nearly tie
        srt = np.sort(want["sims"])
        tau = srt[k - 2]
        near = O.near_threshold(want["sims"], tau)
        rep["mismatches"] = P.check_index_set(gb, wb, lambda i: bool(near[i]), "boundaries")
        rep["near_ties"] = int(near.sum())
    else:
        assert np.array_equal(got["event_offsets"].cpu().numpy(), want["event_offsets"])
        assert np.array_equal(got["frame_event"].cpu().numpy(), want["frame_event"])
    # outputs must be self-consistent whatever the boundaries are
    offs = got["event_offsets"].cpu().numpy()
    assert offs[0] == 0 and offs[-1] == T and np.all(np.diff(offs) >= 1)
    assert np.array_equal(offs[1:-1], gb + 1)
    fe = got["frame_event"].cpu().numpy()
    assert np.array_equal(fe, np.searchsorted(offs, np.arange(T), side="right") - 1)
    return rep


def compress_case(V: np.ndarray, t: np.ndarray, offs: np.ndarray, dtype: str, alpha: float, keep_key: float,
                  keep_nonkey: float, event_agg: int = 0, check_features: bool = True,
                  key_events: Optional[np.ndarray] = None) -> Dict[str, object]:
    T, N, d = V.shape
    want = O.compress_vision(V, t, offs, alpha, keep_key, keep_nonkey, dtype, event_agg, key_events_given=key_events)
    p = B.vision_params(alpha, keep_key, keep_nonkey, event_agg)
    Vd = P.to_torch(V, dtype)
    given = None if key_events is None else torch.from_numpy(np.asarray(key_events).astype(np.uint8)).cuda()
    got = B.metok_compress_vision(Vd, torch.from_numpy(np.asarray(offs, dtype=np.int32)).cuda(),
                                  P.to_torch(t, dtype), p, key_events=given)
    torch.cuda.synchronize()
    rep: Dict[str, object] = {}
    assert int(got["status"].item()) == 0, "device-side wait timed out"
    n_out = int(got["n_out"].item())
    assert n_out == want["n_out"], (n_out, want["n_out"])
    rep["n_out"] = n_out
    ts = got["token_score"].cpu().numpy()
    # scores: relative to the largest |score| of each event segment
    worst = 0.0
    for e in range(len(offs) - 1):
        lo, hi = int(offs[e]) * N, int(offs[e + 1]) * N
        worst = max(worst, P.score_err(ts[lo:hi], want["token_score"][lo:hi]))
    assert worst <= P.TOL[dtype], f"token_score error {worst:.3e}"
    rep["token_score_err"] = worst
    P.check_scores(got["frame_score"].cpu().numpy(), want["frame_score"], dtype, "frame_score")
    P.check_scores(got["event_score"].cpu().numpy(), want["event_score"], dtype, "event_score")
    gk, wk = got["event_is_key"].cpu().numpy(), want["event_is_key"]
    if not np.array_equal(gk, wk):
        es = want["event_score"]
        tau = np.sort(es)[::-1][int(wk.sum()) - 1]
        near = O.near_threshold(es, tau)
        P.check_index_set(np.nonzero(gk)[0], np.nonzero(wk)[0], lambda i: bool(near[i]), "event_is_key")
        rep["event_class_flip"] = True
        return rep                                            # budgets differ downstream: nothing else is comparable
    g_src = got["out_src"][:n_out].cpu().numpy()
    rep["key_near_ties"] = int(want["near_tie"].sum())
    rep["key_mismatches"] = P.check_index_set(g_src, want["out_src"], lambda j: bool(want["near_tie"][j]), "key tokens")
    assert np.all(np.diff(g_src) > 0)
    g_assign = got["assign"].cpu().numpy()
    g_members = got["out_members"][:n_out].cpu().numpy()
    g_event = got["out_event"][:n_out].cpu().numpy()
    tok_event = np.repeat(np.searchsorted(offs, np.arange(T), side="right") - 1, N)
    # validity whatever the near-tie outcome: own event, members add up, keys map to themselves
    assert g_assign.min() >= 0 and g_assign.max() < n_out
    assert np.array_equal(g_event, tok_event[g_src])
    assert np.array_equal(g_event[g_assign], tok_event)
    assert np.array_equal(g_assign[g_src], np.arange(n_out))
    assert np.array_equal(np.bincount(g_assign, minlength=n_out), g_members)
    # assignment parity: compare the key TOKEN each input token joined
    g_key_of = g_src[g_assign]
    w_key_of = want["out_src"][want["assign"]]
    diff = np.nonzero(g_key_of != w_key_of)[0]
    near_assign = want["margin"] < O.NEAR_TIE
    key_flip = rep["key_mismatches"] > 0
    if not key_flip:
        bad = [int(j) for j in diff if not near_assign[j]]
        assert not bad, f"{len(bad)} assignment mismatches outside the near-tie band, e.g. {bad[:8]}"
    rep["assign_near_ties"] = int(near_assign.sum())
    rep["assign_mismatches"] = int(diff.size)
    if check_features:
        # rows whose member sets agree
        same_src = {int(s): i for i, s in enumerate(want["out_src"])}
        touched_w = set(int(s) for s in w_key_of[diff]) | set(int(s) for s in g_key_of[diff])
        rows_g = [i for i, s in enumerate(g_src) if int(s) in same_src and int(s) not in touched_w]
        rows_w = [same_src[int(g_src[i])] for i in rows_g]
        gf = P.to_np(got["out_feats"][:n_out])[rows_g]
        err = P.row_rel_l2(gf, want["out_feats"][rows_w])
        assert err.size > 0.5 * n_out
        assert float(err.max()) <= P.TOL[dtype], f"feature error {float(err.max()):.3e}"
        assert np.array_equal(g_members[rows_g], want["out_members"][rows_w])
        rep["feature_err"] = float(err.max())
        rep["feature_rows_compared"] = int(err.size)
    return rep


def pool_case(V: np.ndarray, t: np.ndarray, offs: np.ndarray, dtype: str, alpha: float, beta: float,
              strides: Sequence[int], event_agg: int = 0, key_frames: Optional[np.ndarray] = None) -> Dict[str, object]:
    """mode POOL (Algorithm 1) against the oracle's adaptive_pool.  Key frames are chosen by frame
    score: a frame whose score is within the near-tie band of its event's cut may flip, and then the
    layouts differ; everything the layout fixes is checked either way."""
    T, N, d = V.shape
    G = int(round(N ** 0.5))
    want = O.adaptive_pool(V, t, offs, alpha, beta, strides, dtype, event_agg, key_frames_given=key_frames)
    p = B.vision_params(alpha, event_agg=event_agg, mode=B.MODE_POOL, beta=beta, s1=strides[0], s2=strides[1],
                        s1_nonkey=strides[2], s2_nonkey=strides[3])
    given = None if key_frames is None else torch.from_numpy(np.asarray(key_frames).astype(np.uint8)).cuda()
    got = B.metok_compress_vision(P.to_torch(V, dtype), torch.from_numpy(np.asarray(offs, dtype=np.int32)).cuda(),
                                  P.to_torch(t, dtype), p, key_frames=given)
    torch.cuda.synchronize()
    rep: Dict[str, object] = {}
    P.check_scores(got["frame_score"].cpu().numpy(), want["frame_score"], dtype, "frame_score")
    assert np.array_equal(got["event_is_key"].cpu().numpy(), want["event_is_key"])
    n_out = int(got["n_out"].item())
    src = got["out_src"][:n_out].cpu().numpy()
    members = got["out_members"][:n_out].cpu().numpy()
    event = got["out_event"][:n_out].cpu().numpy()
    assign = got["assign"].cpu().numpy()
    # layout implied by the outputs themselves: frames in order, windows row-major, every token in one window
    assert np.all(np.diff(src) > 0) and members.min() >= 1 and int(members.sum()) == T * N
    assert np.array_equal(np.bincount(assign, minlength=n_out), members)
    assert np.array_equal(assign[src], np.arange(n_out))
    frame_of = src // N
    assert np.array_equal(event, np.searchsorted(offs, frame_of, side="right") - 1)
    # the stride a frame was pooled with shows in its first window (min(stride, G)^2 cells); strides
    # beyond the grid side all give the one window of the whole frame
    first = np.searchsorted(frame_of, np.arange(T), side="left")
    got_stride = np.rint(np.sqrt(members[first])).astype(np.int32)
    assert np.array_equal(got_stride ** 2, members[first])
    want_stride = np.minimum(want["frame_stride"], G)
    per_frame = np.bincount(frame_of, minlength=T)
    assert np.array_equal(per_frame, (-(-G // got_stride)) ** 2)
    flips = np.nonzero(got_stride != want_stride)[0]
    rep["stride_flips"] = int(flips.size)
    if flips.size:
        fs = want["frame_score"]
        for f in flips:
            e = int(np.searchsorted(offs, f, side="right") - 1)
            seg = fs[int(offs[e]):int(offs[e + 1])]
            nk = int(want["frame_is_key"][int(offs[e]):int(offs[e + 1])].sum())
            tau = np.sort(seg)[::-1][nk - 1]
            assert bool(O.near_threshold(seg, tau)[f - int(offs[e])]), f"frame {f} flipped outside the near-tie band"
        return rep
    assert n_out == want["n_out"]
    assert np.array_equal(frame_of, want["out_frame"])
    err = P.row_rel_l2(P.to_np(got["out_feats"][:n_out]), want["out_feats"])
    assert float(err.max()) <= P.TOL[dtype], f"pooled feature error {float(err.max()):.3e}"
    rep["feature_err"] = float(err.max())
    rep["n_out"] = n_out
    # a window's members: spot-check against the grid arithmetic
    for o in np.linspace(0, n_out - 1, num=min(n_out, 50)).astype(int):
        f = int(frame_of[o]); s_ = int(got_stride[f]); go = -(-G // s_)
        w = o - int(np.searchsorted(frame_of, f, side="left"))
        r0, c0 = (w // go) * s_, (w % go) * s_
        cells = [f * N + r * G + c for r in range(r0, min(G, r0 + s_)) for c in range(c0, min(G, c0 + s_))]
        assert src[o] == cells[0] and members[o] == len(cells)
        assert np.all(assign[cells] == o)
    return rep


def prefill_case(Q: np.ndarray, K: np.ndarray, dtype: str, vis_start: int, n_vis: int, groups: np.ndarray,
                 budgets: Sequence[int], scale: float, hidden: Optional[torch.Tensor] = None) -> Dict[str, object]:
    """`hidden` is a device tensor [S, D] (hash payload) or None."""
    S = K.shape[1]
    want_scores = O.attention_scores(Q, K, vis_start, n_vis, scale)
    want = O.weighted_topk(want_scores, groups, budgets, S, vis_start)
    got = B.metok_prefill_prune(P.to_torch(Q, dtype), P.to_torch(K, dtype), hidden, vis_start, n_vis,
                                torch.from_numpy(np.asarray(groups, dtype=np.int32)).cuda(), budgets, scale)
    torch.cuda.synchronize()
    rep: Dict[str, object] = {}
    assert int(got["status"].item()) == 0, "device-side wait timed out"
    rep["score_err"] = P.check_scores(got["scores"].cpu().numpy(), want_scores, dtype, "attention scores")
    S_out = int(got["S_out"].item())
    assert S_out == want["S_out"], (S_out, want["S_out"])
    keep = got["keep_idx"][:S_out].cpu().numpy()
    assert np.all(np.diff(keep) > 0)
    near = want["near_tie"]
    rep["near_ties"] = int(near.sum())
    rep["mismatches"] = P.check_index_set(
        keep, want["keep_idx"],
        lambda u: vis_start <= u < vis_start + n_vis and bool(near[u - vis_start]), "keep_idx")
    if hidden is not None:
        ho = got["hidden_out"][:S_out]
        # a7 is a pure gather of the rows keep_idx names: bit-exact
        ref = hidden[torch.from_numpy(keep.astype(np.int64)).cuda()]
        assert torch.equal(ho.view(torch.int16) if ho.dtype == torch.bfloat16 else ho,
                           ref.view(torch.int16) if ref.dtype == torch.bfloat16 else ref)
        if rep["mismatches"] == 0:
            rows = np.linspace(0, S_out - 1, num=min(S_out, 64)).astype(np.int64)
            hid_np = P.bits(hidden[torch.from_numpy(want["keep_idx"][rows].astype(np.int64)).cuda()])
            assert np.array_equal(P.bits(ho[torch.from_numpy(rows).cuda()]), hid_np)
    rep["S_out"] = S_out
    return rep


def kv_case(cfg: W.Config, policy: int, layers: Optional[int] = None, per_layer_scores: bool = False,
            l1: int = 3, sample_slabs: int = 12, given_from: Optional[int] = None) -> Dict[str, object]:
    """K/V caches are hash payloads generated on the device; expected rows are
    regenerated on the host from the same hash for the oracle's keep lists."""
    L = cfg.L if layers is None else layers
    n_vis, S_cur = cfg.Nv, cfg.Nv + cfg.kv_text
    dev = torch.device("cuda")
    ks, vs = W.kv_cache_torch(cfg, dev, L)
    scores_np = None
    kwargs = {}
    if policy == O.KV_TOPK:
        scores_np = W.kv_scores(cfg, n_vis, per_layer_scores, L)
        kwargs["scores"] = torch.from_numpy(scores_np).cuda()
        kwargs["keep_ratio"] = cfg.keep_kv
    given = None
    if policy == O.KV_GIVEN:
        rng = np.random.default_rng(given_from or 0)
        given = []
        for layer in range(L):
            n = int(rng.integers(0, S_cur + 1)) if layer else S_cur // 2
            given.append(np.sort(rng.choice(S_cur, size=n, replace=False)).astype(np.int32))
        ki = torch.zeros((L, S_cur), dtype=torch.int32)
        for layer, g in enumerate(given):
            ki[layer, : len(g)] = torch.from_numpy(g)
        kwargs["keep_idx"] = ki.cuda()
        kwargs["keep_len"] = torch.tensor([len(g) for g in given], dtype=torch.int32).cuda()
    want = O.kv_select(policy, L, S_cur, 0, n_vis, l1=l1, keep_ratio=cfg.keep_kv, scores=scores_np, given=given)
    got = B.metok_kv_compact(ks, vs, S_cur, policy, 0, n_vis, l1=l1, **kwargs)
    torch.cuda.synchronize()
    new_len = got["new_len"].cpu().numpy()
    assert int(got["status"].item()) == 0
    assert np.array_equal(new_len, [len(w) for w in want])
    assert np.array_equal(got["keep_len"].cpu().numpy(), new_len)
    keep_idx = got["keep_idx"].cpu().numpy()
    for layer in range(L):
        assert np.array_equal(keep_idx[layer, : new_len[layer]], want[layer]), layer   # scores are tie-free
    # every (layer, K|V, head) slab bit for bit: the payload is regenerated on the device from its hash
    # and gathered with the ORACLE's list
    checked = 0
    for layer in range(L):
        n = int(new_len[layer])
        if n == 0:
            continue
        idx = torch.from_numpy(np.asarray(want[layer], dtype=np.int64)).to(dev)
        for which in (0, 1):
            for head in range(cfg.Hkv):
                src = W.payload_torch(W.kv_salt(cfg, layer, which, head), S_cur, cfg.dh, cfg.dtype, dev)
                t = (vs if which else ks)[layer][head, :n]
                exp = src[idx]
                if cfg.dtype == "bf16":
                    t, exp = t.view(torch.int16), exp.view(torch.int16)
                assert torch.equal(t, exp), (layer, which, head)
                checked += 1
    # a few slabs also against rows regenerated on the host (the numpy form of the hash)
    rng = np.random.default_rng(99)
    slabs = [(int(rng.integers(0, L)), int(rng.integers(0, 2)), int(rng.integers(0, cfg.Hkv)))
             for _ in range(sample_slabs)]
    slabs += [(0, 0, 0), (L - 1, 1, cfg.Hkv - 1)]
    for layer, which, head in slabs:
        n = int(new_len[layer])
        if n == 0:
            continue
        t = (vs if which else ks)[layer][head, :n]
        expect = W.payload_rows_np(W.kv_salt(cfg, layer, which, head), want[layer], cfg.dh, cfg.dtype)
        if cfg.dtype == "bf16":
            assert np.array_equal(P.bits(t), expect), (layer, which, head)
        else:
            assert np.array_equal(t.cpu().numpy(), expect), (layer, which, head)
    return {"kept_rows": int(new_len.sum()), "slabs_checked": checked, "slabs_checked_on_host": len(slabs)}

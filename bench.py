#!/usr/bin/env python
"""Benchmark of the METok hot path on B200.

A "step" is one pass of the whole hot path over a batch of independent synthetic
videos of the 128-frame workload (128 x 144 visual tokens, 28-layer 7B-shaped LLM;
8 videos in flight by default, each on a stream of its own): event
segmentation, stage-1 compression, the three prefill pruning levels at the
sizes the Eq. 6/7 schedule implies, and the KV-cache compaction -- all through
the C ABI.  `value` = visual tokens entering the path per second, inputs resident
in HBM; `e2e` = the same with every step's inputs copied from pinned host memory
and its results copied back inside the timed region.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl reference]

With N > 1 (launched by torch.distributed.run) every rank compresses its own
video: independent replicas, no data-path collective, weak scaling.
"""

from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2506_02850_b200 import workloads as W

EXP_PEAK_GEXP_S = 16 * 148 * 1.965      # exponentials per ns of the whole chip at the maximum SM clock

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

# dram__bytes_read.sum + dram__bytes_write.sum of one video's launches of each kernel, from the committed ncu
# captures (profiles/), keyed by (scope/kernel, workload); a kernel changed since its capture is left out
# (its stage then reports traffic null).
NCU_TRAFFIC_BYTES = {
    ("segment/seg_score_kernel", "frames128"): 136371200,
    ("segment/seg_finish_kernel", "frames128"): 58624,
    ("compress/event_plan_kernel", "frames128"): 131584,
    ("compress/event_topk_kernel", "frames128"): 132352,
    ("compress/merge_assign_mma_kernel", "frames128"): 137563392,
    ("compress/merge_decode_kernel", "frames128"): 279808,
    ("compress/merge_avg_kernel", "frames128"): 147466752,
    ("prefill1/attn_stats_mma_kernel", "frames128"): 19438592,
    ("prefill1/attn_colsum_mma_kernel", "frames128"): 19495680,
    ("prefill1/attn_score_reduce_kernel", "frames128"): 1189120,
    ("prefill1/class_topk_kernel", "frames128"): 217856,
    ("prefill1/gather_rows_kernel", "frames128"): 53984512,
    ("prefill2/attn_stats_mma_kernel", "frames128"): 7494656,
    ("prefill2/attn_colsum_mma_kernel", "frames128"): 7568128,
    ("prefill2/attn_score_reduce_kernel", "frames128"): 442880,
    ("prefill2/class_topk_kernel", "frames128"): 124928,
    ("prefill2/gather_rows_kernel", "frames128"): 15964672,
    ("prefill3/attn_stats_mma_kernel", "frames128"): 2776576,
    ("prefill3/attn_colsum_mma_kernel", "frames128"): 2791936,
    ("prefill3/attn_score_reduce_kernel", "frames128"): 147456,
    ("prefill3/class_topk_kernel", "frames128"): 87808,
    ("prefill3/gather_rows_kernel", "frames128"): 473344,
    ("kv/class_topk_kernel", "frames128"): 139776,
    ("kv/kv_stage_kernel", "frames128"): 4828160,
    ("kv/kv_copy_kernel", "frames128"): 100829184,
}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["_source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["_source"] = "fallback"
    return p


# --------------------------------------------------------------------------- #
# workload
# --------------------------------------------------------------------------- #


def schedule(cfg, B, vis):
    """Per pruning level: class labels and Eq. 6/7 budgets at the sizes the schedule implies."""
    grp_full = W.token_groups(cfg, cfg.Nv, vis=vis)
    N0 = [int((grp_full == 0).sum()), int((grp_full == 1).sum())]
    stages = []
    for stage in range(1, cfg.n_stages + 1):
        if stage == 1:
            groups = grp_full
        else:
            prev = B.metok_retention_budgets(cfg.alpha, cfg.keep_prefill, stage - 1, N0)
            groups = W.token_groups(cfg, int(sum(prev)), n_key=int(prev[0]), stage=stage)
        budgets = B.metok_retention_budgets(cfg.alpha, cfg.keep_prefill, stage, N0)
        stages.append((groups, budgets))
    return stages


PARTS = ("segment", "compress", "prefill", "kv")


class Workload:
    def __init__(self, cfg, device, host_copies: bool, parts=PARTS):
        from paper_2506_02850_b200 import binding as B
        self.B = B
        self.cfg = cfg
        self.dev = device
        self.parts = tuple(parts)
        tdt = torch.float32 if cfg.dtype == "f32" else torch.bfloat16
        vis = W.vision_inputs(cfg)
        self.vis = vis
        self.h = {}                                   # pinned host inputs (e2e only)

        def put(name, arr_or_tensor):
            t = arr_or_tensor if isinstance(arr_or_tensor, torch.Tensor) else torch.from_numpy(np.ascontiguousarray(arr_or_tensor))
            if t.dtype == torch.float32 and tdt == torch.bfloat16 and name not in ("kv_scores",):
                t = t.to(torch.bfloat16)
            if host_copies:
                self.h[name] = t.cpu().pin_memory()
            return t.to(device)

        self.V = put("V", vis["V"])
        self.t = put("t", vis["t"])
        self.params = B.vision_params(cfg.alpha, cfg.keep_enc, cfg.keep_enc)
        self.planted_offsets = torch.from_numpy(np.asarray(vis["event_offsets"], dtype=np.int32)).to(device)
        self.stages = []
        for si, (groups, budgets) in enumerate(schedule(cfg, B, vis) if "prefill" in self.parts else [], start=1):
            pf = W.prefill_inputs(cfg, si, groups.size, groups)
            hidden = W.payload_torch(W.hidden_salt(cfg, si), pf["S"], cfg.D, cfg.dtype, device)
            self.stages.append({
                "Q": put(f"Q{si}", pf["Q"]), "K": put(f"K{si}", pf["K"]),
                "hidden": put(f"hidden{si}", hidden), "groups": put(f"groups{si}", groups.astype(np.int32)),
                "budgets": budgets, "n_vis": int(groups.size), "S": int(pf["S"]),
            })
        self.kv_layers = cfg.L
        self.S_cur = cfg.Nv + cfg.kv_text
        self.ks, self.vs = W.kv_cache_torch(cfg, device) if "kv" in self.parts else ([], [])
        if host_copies:
            self.h["ks"] = [t.cpu().pin_memory() for t in self.ks]
            self.h["vs"] = [t.cpu().pin_memory() for t in self.vs]
        self.kv_scores = torch.from_numpy(W.kv_scores(cfg, cfg.Nv)).to(device)
        self.out = {}
        self.side = None
        self.up = self.down = self.consumed = None     # copy streams of the host-buffer step
        self.scale = float(cfg.dh ** -0.5)

    def twin(self):
        """A second, independent video: the same values in buffers of its own (nothing is shared,
        so it competes for L2 and HBM like any other video would)."""
        import copy
        w = copy.copy(self)
        w.V, w.t = self.V.clone(), self.t.clone()
        w.planted_offsets = self.planted_offsets.clone()
        w.stages = [{k_: (v.clone() if isinstance(v, torch.Tensor) else v) for k_, v in s.items()} for s in self.stages]
        w.ks, w.vs = [x.clone() for x in self.ks], [x.clone() for x in self.vs]
        w.kv_scores = self.kv_scores.clone()
        w.out, w.side, w.h = {}, None, {}
        w.up = w.down = w.consumed = None
        return w

    # one pass of the hot path, device-resident inputs
    def step(self):
        self._segment_compress()
        # The K/V lists need the first level's scores only: the compaction runs on a second stream
        # beside pruning levels 2 and 3 and joins at the end of the step.
        main = torch.cuda.current_stream()
        if self.side is None:
            self.side = torch.cuda.Stream()
        forked = False
        for i in range(len(self.stages)):
            self._prefill_level(i)
            if i == 0 and "kv" in self.parts:
                self.side.wait_stream(main)
                with torch.cuda.stream(self.side):
                    self._kv_call()
                forked = True
        if "kv" in self.parts and not forked:
            self._kv_call()
        if forked:
            main.wait_stream(self.side)

    def _segment_compress(self):
        B, cfg, o = self.B, self.cfg, self.out
        # the text embedding is known before the video is segmented: segmentation and the Eq. 5
        # token scores share one pass over V, and the compressor takes the scores from there
        if "segment" in self.parts:
            B.metok_profile_scope("segment")
            o["seg"] = B.metok_segment_score_events(self.V, cfg.k, self.t, out=o.get("seg"))
        if "compress" in self.parts:
            B.metok_profile_scope("compress")
            offs = o["seg"]["event_offsets"] if "seg" in o else self.planted_offsets
            o["cv"] = B.metok_compress_vision(self.V, offs, self.t, self.params, out=o.get("cv"),
                                              scored=o.get("seg"))

    def _prefill_level(self, i):
        B, o, s = self.B, self.out, self.stages[i]
        B.metok_profile_scope(f"prefill{i + 1}")
        o[f"pf{i}"] = B.metok_prefill_prune(s["Q"], s["K"], s["hidden"], 0, s["n_vis"], s["groups"], s["budgets"],
                                            self.scale, out=o.get(f"pf{i}"))

    def _kv_call(self):
        B, cfg, o = self.B, self.cfg, self.out
        B.metok_profile_scope("kv")
        # KV selection uses the first pruning layer's attention scores (n_vis = all visual tokens)
        scores = o["pf0"]["scores"] if self.stages and self.stages[0]["n_vis"] == cfg.Nv else self.kv_scores
        kv = o.get("kv")
        o["kv"] = B.metok_kv_compact(self.ks, self.vs, self.S_cur, B.KV_TOPK, 0, cfg.Nv, keep_ratio=cfg.keep_kv,
                                     scores=scores, keep_idx=None if kv is None else kv["keep_idx"],
                                     keep_len=None if kv is None else kv["keep_len"],
                                     new_len=None if kv is None else kv["new_len"])

    # the same with host buffers: H2D of every input, D2H of every result
    def e2e_alloc(self):
        self.d2h = {}
        self.step()
        torch.cuda.synchronize()
        o = self.out
        n_out = int(o["cv"]["n_out"].item())
        self.n_out = n_out
        self.d2h["out_feats"] = torch.empty((n_out, self.cfg.d), dtype=self.V.dtype).pin_memory()
        self.d2h["out_src"] = torch.empty(n_out, dtype=torch.int32).pin_memory()
        self.d2h["offsets"] = torch.empty(self.cfg.k + 1, dtype=torch.int32).pin_memory()
        for i, s in enumerate(self.stages):
            so = int(o[f"pf{i}"]["S_out"].item())
            s["S_out"] = so
            self.d2h[f"keep{i}"] = torch.empty(so, dtype=torch.int32).pin_memory()
            self.d2h[f"hidden{i}"] = torch.empty((so, self.cfg.D), dtype=self.V.dtype).pin_memory()
        self.kv_new = int(o["kv"]["new_len"][0].item())
        self.d2h["kv_k"] = [torch.empty((self.cfg.Hkv, self.kv_new, self.cfg.dh), dtype=self.V.dtype).pin_memory()
                            for _ in range(self.kv_layers)]
        self.d2h["kv_v"] = [torch.empty((self.cfg.Hkv, self.kv_new, self.cfg.dh), dtype=self.V.dtype).pin_memory()
                            for _ in range(self.kv_layers)]
        h2d = sum(t.numel() * t.element_size() for k_, t in self.h.items() if isinstance(t, torch.Tensor))
        h2d += sum(t.numel() * t.element_size() for t in self.h["ks"] + self.h["vs"])
        d2h = sum(t.numel() * t.element_size() for k_, t in self.d2h.items() if isinstance(t, torch.Tensor))
        d2h += sum(t.numel() * t.element_size() for t in self.d2h["kv_k"] + self.d2h["kv_v"])
        return h2d, d2h

    def e2e_step(self):
        """Host buffers in, host buffers out.  The uploads run on a copy stream in the order the calls need
        them (frames and text, the pruning levels' inputs, the K/V cache last), each call starts when its
        inputs have landed, and every result goes back on a second copy stream as soon as its call is done:
        the downloads of everything but the compacted cache overlap the upload of the cache."""
        h, o = self.h, self.out
        cur = torch.cuda.current_stream()
        if self.up is None:
            self.up, self.down = torch.cuda.Stream(), torch.cuda.Stream()
        up, down = self.up, self.down
        # the step before has consumed its inputs; its last downloads (the compacted cache) may still run
        # beside this step's first uploads
        if self.consumed is None:
            up.wait_stream(cur)
        else:
            up.wait_event(self.consumed)
        ev = {}
        with torch.cuda.stream(up):
            self.V.copy_(h["V"], non_blocking=True)
            self.t.copy_(h["t"], non_blocking=True)
            ev["vision"] = up.record_event()
            for i, s in enumerate(self.stages, start=1):
                s["Q"].copy_(h[f"Q{i}"], non_blocking=True)
                s["K"].copy_(h[f"K{i}"], non_blocking=True)
                s["hidden"].copy_(h[f"hidden{i}"], non_blocking=True)
                s["groups"].copy_(h[f"groups{i}"], non_blocking=True)
                ev[i] = up.record_event()
            up.wait_stream(down)              # the cache buffers hold the last step's result until it is on the host
            for d, s in zip(self.ks, h["ks"]):
                d.copy_(s, non_blocking=True)
            for d, s in zip(self.vs, h["vs"]):
                d.copy_(s, non_blocking=True)
            ev["kv"] = up.record_event()
        cur.wait_event(ev["vision"])
        self._segment_compress()
        down.wait_stream(cur)
        with torch.cuda.stream(down):
            self.d2h["out_feats"].copy_(o["cv"]["out_feats"][: self.n_out], non_blocking=True)
            self.d2h["out_src"].copy_(o["cv"]["out_src"][: self.n_out], non_blocking=True)
            self.d2h["offsets"].copy_(o["seg"]["event_offsets"], non_blocking=True)
        for i, s in enumerate(self.stages):
            cur.wait_event(ev[i + 1])
            self._prefill_level(i)
            down.wait_stream(cur)
            with torch.cuda.stream(down):
                self.d2h[f"keep{i}"].copy_(o[f"pf{i}"]["keep_idx"][: s["S_out"]], non_blocking=True)
                self.d2h[f"hidden{i}"].copy_(o[f"pf{i}"]["hidden_out"][: s["S_out"]], non_blocking=True)
        cur.wait_event(ev["kv"])
        self._kv_call()
        down.wait_stream(cur)
        with torch.cuda.stream(down):
            for l in range(self.kv_layers):
                self.d2h["kv_k"][l].copy_(self.ks[l][:, : self.kv_new], non_blocking=True)
                self.d2h["kv_v"][l].copy_(self.vs[l][:, : self.kv_new], non_blocking=True)
        self.consumed = cur.record_event()
        cur.wait_stream(down)                 # the step ends when the last result is on the host

    def stage_work(self):
        """Algorithmic work of one video per step of the path: what the method has to move or compute
        (bytes over HBM, tensor flops, exponentials), and the kernels (scope/name of the library's
        brackets) that make up the step."""
        cfg = self.cfg
        b = cfg.elem_bytes
        Nv, d = cfg.Nv, cfg.d
        lens = np.asarray(self.vis["lengths"]) * cfg.N
        k_e = np.array([min(m, max(1, math.ceil(cfg.keep_enc * m - 1e-9))) for m in lens])
        n_out = int(k_e.sum())
        st = {}
        if "segment" in self.parts:
            st["a1+a2 segmentation, text relevance"] = {
                "bound": "hbm", "bytes": float(Nv) * d * b,
                "kernels": ["segment/seg_score_kernel", "segment/seg_finish_kernel", "segment/seg_partial_kernel",
                            "compress/tok_score_kernel", "compress/event_plan_kernel"]}
        if "compress" in self.parts:
            st["a3 key tokens per event"] = {"bound": "latency", "bytes": 8.0 * Nv, "kernels": ["compress/event_topk_kernel"]}
            st["a4 merge-assign, averaging"] = {
                "bound": "tensor+hbm", "flops": float(np.sum(2.0 * (lens - k_e) * k_e * d)),
                "bytes": float(Nv + n_out) * d * b,
                "kernels": ["compress/merge_assign_mma_kernel", "compress/merge_assign_simt_kernel",
                            "compress/merge_decode_kernel", "compress/merge_avg_kernel"]}
        for i, s in enumerate(self.stages, start=1):
            kept = cfg.Lt + sum(min(bg, int((s["groups"] == g).sum().item())) for g, bg in enumerate(s["budgets"]))
            st[f"a5 attention scores, level {i}"] = {
                "bound": "tensor", "flops": 2.0 * 2.0 * cfg.Hq * cfg.Lt * s["S"] * cfg.dh,      # two passes over Q K^T
                "exps": 2.0 * cfg.Hq * cfg.Lt * s["S"], "bytes": float(cfg.Hkv) * s["S"] * cfg.dh * b,
                "kernels": [f"prefill{i}/{k_}" for k_ in ("attn_stats_mma_kernel", "attn_colsum_mma_kernel",
                                                          "attn_stats_kernel", "attn_colsum_kernel",
                                                          "attn_score_reduce_kernel")]}
            st[f"a6 class-wise top-k, level {i}"] = {"bound": "latency", "bytes": 8.0 * s["n_vis"] + 4.0 * kept,
                                                     "kernels": [f"prefill{i}/class_topk_kernel"]}
            st[f"a7 hidden rows, level {i}"] = {"bound": "hbm", "bytes": 2.0 * kept * cfg.D * b,
                                                "kernels": [f"prefill{i}/gather_rows_kernel"]}
        if "kv" in self.parts:
            kv_rows = min(cfg.Nv, math.ceil(cfg.keep_kv * cfg.Nv - 1e-9)) + cfg.kv_text
            st["a8 K/V lists"] = {"bound": "latency", "bytes": 4.0 * Nv + 4.0 * cfg.L * kv_rows,
                                  "kernels": ["kv/class_topk_kernel", "kv/kv_paper_lists_kernel", "kv/kv_check_lists_kernel"]}
            st["a9 K/V in-place gather"] = {"bound": "hbm", "bytes": 2.0 * kv_rows * cfg.dh * b * 2 * cfg.Hkv * cfg.L,
                                            "kernels": ["kv/kv_stage_kernel", "kv/kv_copy_kernel", "kv/kv_gather_kernel"]}
        return st


# --------------------------------------------------------------------------- #
# clocks
# --------------------------------------------------------------------------- #


class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.f = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.proc is None:
            return out
        try:
            self.proc.terminate()
            self.proc.wait(timeout=5)
            self.f.close()
            rows = [r.strip().split(",") for r in open(self.path) if r.strip()]
            os.unlink(self.path)
            sm = [float(r[0]) for r in rows if len(r) >= 6]
            if sm:
                out["sm_mhz"] = float(np.median(sm))
                out["sm_max_mhz"] = float(rows[0][1])
                names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
                for j, n in enumerate(names):
                    if any(r[2 + j].strip().lower().startswith("active") for r in rows if len(r) >= 6):
                        out["reasons"].append(n)
                out["samples"] = len(sm)
        except Exception:
            pass
        return out


# --------------------------------------------------------------------------- #
# CPU baseline: the oracle, as it stands, on a bounded sample of the workload
# --------------------------------------------------------------------------- #


def oracle_sample_step(cfg, sample):
    """One pass of the oracle over the sample."""
    from oracle import metok_oracle as O
    V, t, offs, levels, kv = sample
    O.segment_events(V, len(offs) - 1)
    O.compress_vision(V, t, offs, cfg.alpha, cfg.keep_enc, cfg.keep_enc, cfg.dtype)
    first = None
    for groups, budgets, Q, K, hidden in levels:
        pr = O.prefill_prune(Q, K, hidden, 0, groups.size, groups, budgets, cfg.dh ** -0.5)
        first = pr if first is None else first
    lists = O.kv_select(O.KV_TOPK, len(kv[0]), kv[0][0].shape[1], 0, levels[0][0].size, keep_ratio=cfg.keep_kv,
                        scores=first["scores"])
    O.kv_compact(kv[0], kv[1], lists)


def oracle_sample(cfg, kv_layers=4):
    """The whole video through segmentation, stage-1 compression and every pruning level; the K/V
    compaction on `kv_layers` of the layers (building all of them on the host takes minutes)."""
    from oracle import metok_oracle as O
    vis = W.vision_inputs(cfg)
    grp_full = W.token_groups(cfg, cfg.Nv, vis=vis)
    N0 = [int((grp_full == 0).sum()), int((grp_full == 1).sum())]
    levels = []
    for stage in range(1, cfg.n_stages + 1):
        if stage == 1:
            groups = grp_full
        else:
            prev = O.retention_budgets(cfg.alpha, cfg.keep_prefill, stage - 1, N0)
            groups = W.token_groups(cfg, int(prev.sum()), n_key=int(prev[0]), stage=stage)
        budgets = O.retention_budgets(cfg.alpha, cfg.keep_prefill, stage, N0).tolist()
        pf = W.prefill_inputs(cfg, stage, groups.size, groups)
        hidden = W.payload_rows_np(W.hidden_salt(cfg, stage), np.arange(pf["S"]), cfg.D, cfg.dtype)
        levels.append((groups, budgets, pf["Q"], pf["K"], hidden))
    kv_layers = min(kv_layers, cfg.L)
    S = cfg.Nv + cfg.kv_text
    kv = tuple([np.stack([W.payload_rows_np(W.kv_salt(cfg, l, w, h), np.arange(S), cfg.dh, cfg.dtype)
                          for h in range(cfg.Hkv)]) for l in range(kv_layers)] for w in (0, 1))
    what = (f"all {cfg.T} frames ({cfg.Nv} visual tokens): segmentation, stage-1 compression, "
            f"{cfg.n_stages} pruning levels, KV TOPK compaction of {kv_layers} of {cfg.L} layers")
    return (vis["V"], vis["t"], vis["event_offsets"], levels, kv), cfg.Nv, what


def cpu_threads():
    try:
        from threadpoolctl import threadpool_info
        n = max([i.get("num_threads", 1) for i in threadpool_info()] + [1])
        return int(n)
    except Exception:
        return os.cpu_count() or 1


def first_frames(cfg, frames):
    """The same workload cut to its first `frames` frames (events in proportion, at least two frames each)."""
    import dataclasses
    if frames >= cfg.T:
        return cfg
    k = max(1, min(cfg.k, (cfg.k * frames) // cfg.T, frames // 2))
    return dataclasses.replace(cfg, T=frames, k=k, events="compose")


def time_oracle(cfg, steps, warmup, budget_s=None):
    """Tokens per second of the oracle over `steps` passes.  With a time budget the pass runs on the
    first frames of the video only, as many as fit: the cost per frame comes from one pass over eight."""
    if budget_s is not None:
        probe = first_frames(cfg, min(cfg.T, 8))
        sample, _, _ = oracle_sample(probe)
        t0 = time.perf_counter()
        oracle_sample_step(probe, sample)
        per_frame = (time.perf_counter() - t0) / probe.T
        # the cost grows faster than the frame count (events get longer): half of what a linear estimate allows
        frames = int(0.5 * budget_s / max(steps + warmup, 1) / max(per_frame, 1e-9))
        full_T = cfg.T
        cfg = first_frames(cfg, max(2, min(cfg.T, frames)))
    sample, n_tok, what = oracle_sample(cfg)
    if budget_s is not None and cfg.T < full_T:
        what = what.replace(f"all {cfg.T} frames", f"the first {cfg.T} of {full_T} frames, {cfg.k} events")
    for _ in range(warmup):
        oracle_sample_step(cfg, sample)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle_sample_step(cfg, sample)
    dt = (time.perf_counter() - t0) / max(steps, 1)
    return n_tok / dt, dt, what


# --------------------------------------------------------------------------- #


def chained_run(cfg, dev, B, timed):
    """The four calls fed by one another: segmentation -> stage-1 compression -> the pruning levels on the
    survivors -> K/V compaction of the cache the survivors would have left.  Q, K and hidden rows of a
    level are gathered (torch.index_select, inside the timed region) from per-token synthetic tensors by
    the original ids of the tokens still alive; the layers of the model that would sit in between are not
    part of the path.  Sizes are those of the first, untimed pass (the inputs are fixed, so they repeat)."""
    tdt = torch.float32 if cfg.dtype == "f32" else torch.bfloat16
    vis = W.vision_inputs(cfg)
    V = torch.from_numpy(vis["V"]).to(tdt).to(dev)
    t = torch.from_numpy(vis["t"]).to(tdt).to(dev)
    params = B.vision_params(cfg.alpha, cfg.keep_enc, cfg.keep_enc)
    grp_full = torch.from_numpy(W.token_groups(cfg, cfg.Nv, vis=vis).astype(np.int32)).to(dev)
    full = []
    for s_ in range(1, cfg.n_stages + 1):
        pf = W.prefill_inputs(cfg, s_, cfg.Nv, W.token_groups(cfg, cfg.Nv, vis=vis))
        full.append({"Q": torch.from_numpy(pf["Q"]).to(tdt).to(dev), "K": torch.from_numpy(pf["K"]).to(tdt).to(dev),
                     "hidden": W.payload_torch(W.hidden_salt(cfg, s_), cfg.Nv + cfg.Lt, cfg.D, cfg.dtype, dev)})
    text_rows = torch.arange(cfg.Nv, cfg.Nv + cfg.Lt, device=dev, dtype=torch.int64)
    seg = B.metok_segment_score_events(V, cfg.k, t)
    cv = B.metok_compress_vision(V, seg["event_offsets"], t, params, scored=seg)
    torch.cuda.synchronize()
    n1 = int(cv["n_out"].item())
    g1 = grp_full[cv["out_src"][:n1].long()]
    N0 = [int((g1 == 0).sum().item()), int((g1 == 1).sum().item())]
    sizes = B.metok_prune_schedule_sizes(cfg.n_stages, cfg.alpha, cfg.keep_prefill, N0)
    bufs = [{"K": torch.empty((cfg.Hkv, sizes[i] + cfg.Lt, cfg.dh), dtype=tdt, device=dev),
             "hidden": torch.empty((sizes[i] + cfg.Lt, cfg.D), dtype=tdt, device=dev)} for i in range(cfg.n_stages)]
    budgets = [B.metok_retention_budgets(cfg.alpha, cfg.keep_prefill, i + 1, N0) for i in range(cfg.n_stages)]
    S_kv = n1 + cfg.kv_text
    ks = [W.payload_torch(W.kv_salt(cfg, l, 0, 0), cfg.Hkv * S_kv, cfg.dh, cfg.dtype, dev).view(cfg.Hkv, S_kv, cfg.dh)
          for l in range(cfg.L)]
    vs = [W.payload_torch(W.kv_salt(cfg, l, 1, 0), cfg.Hkv * S_kv, cfg.dh, cfg.dtype, dev).view(cfg.Hkv, S_kv, cfg.dh)
          for l in range(cfg.L)]
    out = {}
    scale = float(cfg.dh ** -0.5)

    def chained_step():
        out["seg"] = B.metok_segment_score_events(V, cfg.k, t, out=out.get("seg"))
        out["cv"] = B.metok_compress_vision(V, out["seg"]["event_offsets"], t, params, out=out.get("cv"), scored=out["seg"])
        idx = out["cv"]["out_src"][:n1].long()
        grp = grp_full[idx]
        for i in range(cfg.n_stages):
            rows = torch.cat([idx, text_rows])
            torch.index_select(full[i]["K"], 1, rows, out=bufs[i]["K"])
            torch.index_select(full[i]["hidden"], 0, rows, out=bufs[i]["hidden"])
            pf = B.metok_prefill_prune(full[i]["Q"], bufs[i]["K"], bufs[i]["hidden"], 0, sizes[i], grp.contiguous(),
                                       budgets[i], scale, out=out.get(f"pf{i}"))
            out[f"pf{i}"] = pf
            if i == 0:
                kv = out.get("kv")
                out["kv"] = B.metok_kv_compact(ks, vs, S_kv, B.KV_TOPK, 0, n1, keep_ratio=cfg.keep_kv, scores=pf["scores"],
                                               keep_idx=None if kv is None else kv["keep_idx"],
                                               keep_len=None if kv is None else kv["keep_len"],
                                               new_len=None if kv is None else kv["new_len"])
            keepv = pf["keep_idx"][: sizes[i + 1]].long()        # the visual survivors come first (vis_start = 0)
            idx, grp = idx[keepv], grp[keepv]

    chained_step()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        chained_step()

    def chained_graph():
        g.replay()

    steps = 200
    ms = timed(chained_graph, steps) / steps
    return {"ms_per_video": ms, "tokens_per_s": cfg.Nv / (ms * 1e-3), "n_out": n1, "level_sizes": sizes,
            "kv_rows_before": S_kv, "launch": "cuda_graph",
            "what": "segment -> compress -> pruning levels on the survivors -> K/V compaction, one video alone; "
                    "includes the torch gathers that stand in for the model's layers between the calls"}


def unplanted_attention_run(cfg, dev, B, timed):
    """Pruning level 1 at full size on Q/K without the planted relevance: every score then lies inside the
    near-tie band of the cut (nothing to compare index by index), but the work is the same."""
    tdt = torch.float32 if cfg.dtype == "f32" else torch.bfloat16
    vis = W.vision_inputs(cfg)
    groups = W.token_groups(cfg, cfg.Nv, vis=vis)
    N0 = [int((groups == 0).sum()), int((groups == 1).sum())]
    budgets = B.metok_retention_budgets(cfg.alpha, cfg.keep_prefill, 1, N0)
    pf = W.prefill_inputs(cfg, 1, cfg.Nv, groups, planted=False)
    Q, K = torch.from_numpy(pf["Q"]).to(tdt).to(dev), torch.from_numpy(pf["K"]).to(tdt).to(dev)
    hidden = W.payload_torch(W.hidden_salt(cfg, 1), pf["S"], cfg.D, cfg.dtype, dev)
    grp = torch.from_numpy(groups.astype(np.int32)).to(dev)
    out = {}

    def call():
        out["pf"] = B.metok_prefill_prune(Q, K, hidden, 0, cfg.Nv, grp, budgets, float(cfg.dh ** -0.5), out=out.get("pf"))

    call()
    torch.cuda.synchronize()
    sc = out["pf"]["scores"].float()
    spread = float((sc.max() - sc.min()) / sc.mean())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        call()

    def unplanted_graph():
        g.replay()

    ms = timed(unplanted_graph, 200) / 200
    return {"ms_per_call": ms, "relative_score_spread": spread, "S_out": int(out["pf"]["S_out"].item()),
            "what": "metok_prefill_prune, level 1, all visual tokens, Q/K ~ N(0, 1/sqrt(dh)) only"}


def max_over_ranks(ms: float, dist, device) -> float:
    """The slowest rank's time: replicas finish together only when the last one does."""
    if dist is None:
        return float(ms)
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def replica_throughput(tokens_per_replica: int, world: int, ms_per_step: float) -> float:
    """Whole-job tokens/s of `world` independent replicas that each finish a step in ms_per_step."""
    return world * tokens_per_replica / (ms_per_step * 1e-3)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--config", default="frames128")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="time eager launches instead of a CUDA graph of the step")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="skip the chained run and the run without planted relevance")
    ap.add_argument("--no-sustain", action="store_true",
                    help="time exactly --steps steps (for profiler captures, where a one-second region is thousands of launches)")
    ap.add_argument("--videos", type=int, default=8,
                    help="independent videos in flight per step, each on a stream of its own (a step = this batch)")
    ap.add_argument("--parts", default=",".join(PARTS),
                    help="comma-separated subset of the four calls (for profiler captures that should hold little "
                         "memory); anything but the full list is not a benchmark result")
    args = ap.parse_args()
    cfg = W.CONFIGS[args.config]
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    workload_name = (f"{cfg.name}: {cfg.T} frames x {cfg.N} tokens, d={cfg.d} {cfg.dtype}, k={cfg.k} events, "
                     f"{cfg.Lt} text tokens, {cfg.Hq}/{cfg.Hkv} heads dh={cfg.dh}, hidden {cfg.D}, "
                     f"{cfg.n_stages} pruning levels, {cfg.L}-layer K/V cache, keep {cfg.keep_enc}/{cfg.keep_prefill}/{cfg.keep_kv}")

    if args.impl == "reference":
        # the oracle on the host cores; rank 0 alone
        if rank != 0:
            return
        W_ = max(args.warmup, 0)
        val, dt, what = time_oracle(cfg, args.steps, min(W_, 1), budget_s=150.0)   # the whole run within a few minutes
        line = {"impl": "reference", "metric": "visual_tokens_per_s", "value": val, "unit": "tokens/s",
                "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3,
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
                "data": "synthetic", "config": {"workload": workload_name},
                "cpu_baseline": {"value": val, "unit": "tokens/s", "cores": cpu_threads(), "kind": "oracle",
                                 "sample": what},
                "e2e": {"value": val, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
        print(json.dumps(line))
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the METok hot path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist_
        dist = dist_
        dist.init_process_group("nccl", device_id=dev)

    from paper_2506_02850_b200 import binding as B
    B.lib()
    parts = tuple(p for p in args.parts.split(",") if p)
    assert all(p in PARTS for p in parts), parts
    partial = set(parts) != set(PARTS)
    if partial:
        args.no_e2e = True
    wl = Workload(cfg, dev, host_copies=not args.no_e2e, parts=parts)
    n_videos = max(1, args.videos)
    wls = [wl] + [wl.twin() for _ in range(n_videos - 1)]
    # Every video's own chain of calls is its critical path; the K/V compaction beside pruning levels 2-3 is
    # not.  The videos' streams get the higher priority, so that a waiting kernel of a chain goes ahead of the
    # compaction's remaining CTAs when an SM has room.
    lanes = [torch.cuda.Stream(priority=-1) for _ in range(n_videos - 1)]
    capture_stream = torch.cuda.Stream(priority=-1)
    warm = max(args.warmup, 3)

    def batch_step():
        """All videos of the batch, each on its own stream, joined at the end."""
        main = torch.cuda.current_stream()
        for st in lanes:
            st.wait_stream(main)
        wls[0].step()
        for w, st in zip(wls[1:], lanes):
            with torch.cuda.stream(st):
                w.step()
        for st in lanes:
            main.wait_stream(st)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    host_ms = {}

    def timed(fn, steps):
        for _ in range(warm):
            fn()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        t0 = time.perf_counter()
        for _ in range(steps):
            fn()
        host_ms[fn.__name__] = (time.perf_counter() - t0) * 1e3 / steps     # time to enqueue one step
        e1.record()
        barrier()
        return max_over_ranks(e0.elapsed_time(e1), dist, dev)

    # eager: every step issues its C-ABI calls from Python
    eager_ms_per_step = timed(batch_step, min(args.steps, 50)) / min(args.steps, 50)
    # the same calls captured once in a CUDA graph and replayed: the calls enqueue on a stream
    # and never synchronise, so one capture of a step holds all of its launches
    graph = graph_one = None
    if not args.no_graph:
        graph_one = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph_one, stream=capture_stream):
            wl.step()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=capture_stream):
            batch_step()

        def step_graph():
            graph.replay()

        def step_graph_one():
            graph_one.replay()
    run_one = step_graph_one if graph_one is not None else wl.step
    run_batch = step_graph if graph is not None else batch_step
    # latency of one video alone on the GPU
    ms_one_video = timed(run_one, min(args.steps, 200)) / min(args.steps, 200)
    # exactly --steps steps (a burst when that is a few milliseconds) ...
    burst_ms = timed(run_batch, args.steps) / args.steps
    # ... and the sustained figure: as many steps as fill at least a second (and no fewer than --steps),
    # the clocks sampled meanwhile; `value` is this one, whatever --steps was
    sustain_steps = args.steps if args.no_sustain else max(args.steps, int(math.ceil(1000.0 / max(burst_ms, 1e-3))))
    sampler = ClockSampler(local)
    sampler.start()
    total_ms = timed(run_batch, sustain_steps)
    clocks = sampler.stop()
    ms_per_step = total_ms / sustain_steps
    value = replica_throughput(cfg.Nv * n_videos, world, ms_per_step)

    # per-kernel times: one video's step with the library's event brackets on.  Captured in a CUDA
    # graph the brackets are event-record nodes, so a replay times the kernels as they run in the
    # timed region (no host launch gap inside a bracket); eager launches otherwise.
    barrier()
    prof_steps = max(1, min(args.steps, 100))
    B.metok_profile_begin()
    if not args.no_graph:
        graph_prof = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph_prof):
            wl.step()
        prof = {}
        for _ in range(prof_steps):
            graph_prof.replay()
            torch.cuda.synchronize()
            for k_, v in B.metok_profile_read().items():
                ent = prof.setdefault(k_, {"launches": 0, "ms": 0.0})
                ent["launches"] += v["launches"]
                ent["ms"] += v["ms"]
        del graph_prof
        B.metok_profile_end()
    else:
        for _ in range(prof_steps):
            wl.step()
        prof = B.metok_profile_end()
    B.metok_profile_scope(None)
    launches_per_step = sum(v["launches"] for v in prof.values()) // prof_steps
    peaks = load_peaks()
    hbm_peak, tc_peak = float(peaks["hbm_gbs"]), float(peaks["bf16_tflops_sustained"])
    kern_us = {k_: v["ms"] * 1e3 / prof_steps for k_, v in prof.items()}
    # every bracket costs the same few microseconds on top of its kernel (two event nodes): what the
    # brackets add up to beyond the step's own time, per launch
    bracket_us = (max(0.0, sum(kern_us.values()) - ms_one_video * 1e3) / max(1, launches_per_step)
                  if not partial else None)

    # the steps of the path: algorithmic work / the summed time of ALL kernels a step launches
    stages = {}
    for name, w_ in wl.stage_work().items():
        ks = [k_ for k_ in w_["kernels"] if k_ in kern_us]
        if not ks:
            continue
        us = sum(kern_us[k_] for k_ in ks)
        ent = {"us": round(us, 2), "kernels": {k_.split("/", 1)[1]: round(kern_us[k_], 2) for k_ in ks},
               "launches": sum(prof[k_]["launches"] for k_ in ks) // prof_steps, "bound": w_["bound"]}
        traffic = [NCU_TRAFFIC_BYTES.get((k_, cfg.name)) for k_ in ks]
        ent["traffic"] = None if any(t is None for t in traffic) else float(sum(traffic))
        if "bytes" in w_:
            ent["algorithmic_bytes"] = w_["bytes"]
            ent["GB/s"] = round(w_["bytes"] / (us * 1e-6) / 1e9, 1)
            ent["frac_hbm"] = round(ent["GB/s"] / hbm_peak, 4)
        if "flops" in w_:
            ent["algorithmic_flops"] = w_["flops"]
            ent["TFLOP/s"] = round(w_["flops"] / (us * 1e-6) / 1e12, 1)
            ent["frac_tensor"] = round(ent["TFLOP/s"] / tc_peak, 4)
        if "exps" in w_:
            ent["exponentials"] = w_["exps"]
            ent["Gexp/s"] = round(w_["exps"] / (us * 1e-6) / 1e9, 1)
            # the special-function unit gives 16 ex2.approx results per clock and SM (measured with a
            # register-only kernel; the packed half-precision form gives the same 16 results per clock)
            ent["frac_exp"] = round(ent["Gexp/s"] / EXP_PEAK_GEXP_S, 4)
        # fraction of the binding roof: the slower of the HBM and the tensor floor over the measured time
        if w_["bound"] != "latency":
            ent["frac"] = max(ent.get("frac_hbm", 0.0), ent.get("frac_tensor", 0.0)) if w_["bound"] == "tensor+hbm" else (
                ent.get("frac_tensor") if w_["bound"] == "tensor" else ent.get("frac_hbm"))
        stages[name] = ent

    # the headline roofline entry: the kernel with the largest share among those that stream data or run
    # on the tensor cores (the one-SM selection launches are latency-bound: an HBM fraction says nothing)
    def kernel_entry(full_name, us, bound, units):
        if bound == "tensor":
            ach, peak, unit = units / (us * 1e-6) / 1e12, tc_peak, "TFLOP/s"
        else:
            ach, peak, unit = units / (us * 1e-6) / 1e9, hbm_peak, "GB/s"
        return {"kernel": full_name.split("/", 1)[-1], "scope": full_name.split("/", 1)[0], "bound": bound,
                "achieved": ach, "peak": peak, "unit": unit, "frac": ach / peak,
                "peak_source": peaks["_source"] + " (HBM copy; bf16 sustained)",
                "traffic": NCU_TRAFFIC_BYTES.get((full_name, cfg.name)), "us_per_launch": us}
    kernel_work = {}
    sw = wl.stage_work()
    def put_work(kname, bound, units):
        if kname in kern_us:
            kernel_work[kname] = (bound, units)
    if "a4 merge-assign, averaging" in sw:
        a4 = sw["a4 merge-assign, averaging"]
        put_work("compress/merge_assign_mma_kernel", "tensor", a4["flops"])
        put_work("compress/merge_assign_simt_kernel", "tensor", a4["flops"])
        put_work("compress/merge_avg_kernel", "hbm", a4["bytes"])
    if "a1+a2 segmentation, text relevance" in sw:
        put_work("segment/seg_score_kernel", "hbm", sw["a1+a2 segmentation, text relevance"]["bytes"])
    for i in range(1, len(wl.stages) + 1):
        a5, a7 = sw[f"a5 attention scores, level {i}"], sw[f"a7 hidden rows, level {i}"]
        for k_ in ("attn_stats_mma_kernel", "attn_colsum_mma_kernel", "attn_stats_kernel", "attn_colsum_kernel"):
            put_work(f"prefill{i}/{k_}", "tensor", a5["flops"] / 2)
        put_work(f"prefill{i}/gather_rows_kernel", "hbm", a7["bytes"])
    if "a9 K/V in-place gather" in sw:
        put_work("kv/kv_copy_kernel", "hbm", sw["a9 K/V in-place gather"]["bytes"])
    roofline = None
    if kernel_work:
        top = max(kernel_work, key=lambda k_: kern_us[k_])
        roofline = kernel_entry(top, kern_us[top], *kernel_work[top])
        roofline["per_kernel"] = {k_: dict(us=round(kern_us[k_], 2), **{kk: (round(vv, 4) if isinstance(vv, float) else vv)
                                                                        for kk, vv in kernel_entry(k_, kern_us[k_], *kernel_work[k_]).items()
                                                                        if kk in ("bound", "achieved", "unit", "frac")})
                                  for k_ in sorted(kernel_work, key=lambda k_: -kern_us[k_])}
        roofline["latency_bound_kernels_us"] = {k_: round(u, 2) for k_, u in sorted(kern_us.items(), key=lambda kv: -kv[1])
                                                if k_ not in kernel_work}
        roofline["bracket_overhead_us_per_launch"] = bracket_us

    # one video against its own floors: the algorithmic HBM bytes and tensor flops of all steps
    step_roofline = None
    if not partial:
        tot_bytes = sum(w_.get("bytes", 0.0) for n_, w_ in sw.items() if w_["bound"] in ("hbm", "tensor+hbm"))
        tot_bytes += sum(w_.get("bytes", 0.0) for n_, w_ in sw.items() if w_["bound"] == "tensor")      # K read by the scoring
        tot_flops = sum(w_.get("flops", 0.0) for w_ in sw.values())
        floor_us = tot_bytes / (hbm_peak * 1e9) * 1e6
        tensor_us = tot_flops / (tc_peak * 1e12) * 1e6
        step_roofline = {"algorithmic_bytes": tot_bytes, "algorithmic_flops": tot_flops, "hbm_floor_us": round(floor_us, 1),
                         "tensor_floor_us": round(tensor_us, 1),
                         "one_video_alone": {"us": round(ms_one_video * 1e3, 1), "frac_of_hbm_floor": round(floor_us / (ms_one_video * 1e3), 3)},
                         "per_video_in_batch": {"us": round(ms_per_step * 1e3 / n_videos, 1),
                                                "frac_of_hbm_floor": round(floor_us / (ms_per_step * 1e3 / n_videos), 3)}}

    extras = {}
    if not partial and rank == 0 and world == 1 and not args.no_extras:
        extras["chained"] = chained_run(cfg, dev, B, timed)
        extras["no_planted_relevance"] = unplanted_attention_run(cfg, dev, B, timed)

    e2e = None
    if not args.no_e2e:
        h2d, d2h = wl.e2e_alloc()
        e2e_steps = max(3, min(args.steps, 10))
        ms = timed(wl.e2e_step, e2e_steps) / e2e_steps
        e2e = {"value": replica_throughput(cfg.Nv, world, ms), "unit": "tokens/s", "ms_per_step": ms,
               "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "steps": e2e_steps}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        v, dt, what = time_oracle(cfg, 3, 1)
        cpu = {"value": v, "unit": "tokens/s", "cores": cpu_threads(), "kind": "oracle", "sample": what,
               "seconds": dt}
        try:
            from threadpoolctl import threadpool_limits
            with threadpool_limits(limits=1):
                v1, dt1, _ = time_oracle(cfg, 1, 0)
            cpu["one_thread"] = {"value": v1, "seconds": dt1, "cores": 1}
        except Exception as exc:                       # the limit is a convenience of the numpy build
            cpu["one_thread"] = {"unavailable": str(exc)}

    if rank == 0:
        line = {"metric": "visual_tokens_per_s", "value": value, "unit": "tokens/s", "n_gpus": world,
                "steps": args.steps, "warmup": warm, "ms_per_step": ms_per_step, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
                "config": {"workload": workload_name, "l2": "inputs larger than L2 (V 132 MB, hidden 133 MB, K/V 1.06 GB touched between reuses)",
                           "videos_in_flight": n_videos, "parallelism": f"replicas x{world}"},
                "timed_steps": sustain_steps, "burst": {"steps": args.steps, "ms_per_step": burst_ms,
                                                        "value": replica_throughput(cfg.Nv * n_videos, world, burst_ms)},
                "single_video": {"ms_per_video": ms_one_video, "tokens_per_s": replica_throughput(cfg.Nv, world, ms_one_video)},
                "launch": "cuda_graph" if graph is not None else "eager", "eager_ms_per_step": eager_ms_per_step,
                "host_enqueue_ms_per_step": host_ms.get("batch_step"), "clocks": clocks, "e2e": e2e,
                "gpu_launches": launches_per_step * n_videos * sustain_steps,
                "roofline": roofline, "stages": stages, "step_roofline": step_roofline, "cpu_baseline": cpu}
        line.update(extras)
        if partial:
            line["partial"] = "only " + ",".join(parts) + ": not a benchmark result"
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

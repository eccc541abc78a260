"""Thin ctypes binding of ``libmetok.so``: argument marshalling only.

Every function here has the name of the C entry point it calls
(``include/metok.h``), allocates the output tensors and the workspace with
torch, passes raw device pointers and the current CUDA stream, and returns the
outputs.  Nothing is computed in Python and there is no fallback: if the
library is missing, or a call returns an error status, an exception is raised.
"""

from __future__ import annotations

import ctypes
import os
from typing import Dict, List, Optional, Sequence

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "lib", "libmetok.so")

F32, BF16 = 0, 1
SIM_FLATTEN, SIM_MEANPOOL = 0, 1
AGG_MEAN, AGG_MAX = 0, 1
MODE_TOPK_MERGE, MODE_POOL = 0, 1
KV_PAPER, KV_TOPK, KV_GIVEN = 0, 1, 2

_c = ctypes
_vp, _i, _sz, _f, _d = _c.c_void_p, _c.c_int, _c.c_size_t, _c.c_float, _c.c_double


class VisionParams(_c.Structure):
    _fields_ = [("alpha", _d), ("event_agg", _i), ("mode", _i), ("keep_key", _d), ("keep_nonkey", _d),
                ("beta", _d), ("s1", _i), ("s2", _i), ("s1_nonkey", _i), ("s2_nonkey", _i),
                ("token_inv_norm", _vp), ("key_events_given", _vp), ("key_frames_given", _vp)]


class PruneLevel(_c.Structure):
    _fields_ = [("q_text", _vp), ("k_all", _vp), ("hidden", _vp), ("hidden_out", _vp), ("scores", _vp),
                ("keep_idx", _vp), ("S_out", _vp), ("token_group", _vp), ("origin", _vp)]


class MetokError(RuntimeError):
    def __init__(self, fn: str, status: int, text: str, cuda_error: int = 0):
        self.status = status
        self.cuda_error = cuda_error
        extra = f" (cudaError {cuda_error})" if cuda_error else ""
        super().__init__(f"{fn} failed: {status} {text}{extra}")


_SIGNATURES = {
    "metok_segment_events_workspace_bytes": (_sz, [_i, _i, _i, _i, _i]),
    "metok_segment_events": (_i, [_vp, _i, _i, _i, _i, _i, _i, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "metok_segment_events_static_capacity": (_sz, []),
    "metok_segment_events_static": (_i, [_vp, _i, _i, _i, _i, _i, _i, _vp, _vp, _vp, _vp, _vp]),
    "metok_segment_score_events_workspace_bytes": (_sz, [_i, _i, _i, _i]),
    "metok_segment_score_events": (_i, [_vp, _i, _i, _i, _i, _i, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "metok_compress_vision_bound": (_i, [_i, _i, _i, _c.POINTER(VisionParams)]),
    "metok_compress_vision_workspace_bytes": (_sz, [_i, _i, _i, _i, _i, _i, _c.POINTER(VisionParams)]),
    "metok_compress_vision": (_i, [_vp, _i, _i, _i, _i, _vp, _i, _vp, _c.POINTER(VisionParams),
                                   _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i, _vp, _sz, _vp]),
    "metok_prefill_prune_workspace_bytes": (_sz, [_i, _i, _i, _i, _i, _i, _i]),
    "metok_prefill_prune": (_i, [_vp, _vp, _vp, _i, _i, _i, _i, _i, _i, _i, _i, _i, _vp, _i,
                                 _c.POINTER(_c.c_int32), _f, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "metok_attention_scores": (_i, [_vp, _vp, _i, _i, _i, _i, _i, _i, _i, _i, _f, _i, _vp, _vp, _sz, _vp]),
    "metok_prune_by_scores_workspace_bytes": (_sz, []),
    "metok_prune_by_scores": (_i, [_vp, _vp, _i, _i, _i, _i, _i, _vp, _i, _c.POINTER(_c.c_int32), _vp, _vp, _vp,
                                   _vp, _sz, _vp]),
    "metok_retention_budgets": (_i, [_d, _d, _i, _c.POINTER(_c.c_int32), _c.POINTER(_c.c_int32)]),
    "metok_prune_schedule_sizes": (_i, [_i, _d, _d, _c.POINTER(_c.c_int32), _c.POINTER(_c.c_int32)]),
    "metok_prefill_prune_schedule_workspace_bytes": (_sz, [_i, _i, _i, _i, _i, _i, _i, _i, _d, _d,
                                                          _c.POINTER(_c.c_int32)]),
    "metok_prefill_prune_schedule": (_i, [_c.POINTER(PruneLevel), _i, _i, _i, _i, _i, _i, _i, _i, _i, _i, _d, _d,
                                          _c.POINTER(_c.c_int32), _f, _vp, _vp, _sz, _vp]),
    "metok_kv_compact_workspace_bytes": (_sz, [_i, _i, _i, _i, _i, _i, _i]),
    "metok_kv_compact": (_i, [_c.POINTER(_vp), _c.POINTER(_vp), _i, _i, _i, _i, _i, _i, _i, _i, _d, _i, _i,
                              _vp, _i, _vp, _vp, _vp, _vp, _sz, _vp]),
    "metok_profile_begin": (_i, []),
    "metok_profile_read": (_i, [_c.c_char_p, _sz]),
    "metok_profile_end": (_i, [_c.c_char_p, _sz]),
    "metok_profile_scope": (_i, [_c.c_char_p]),
    "metok_prune_schedule_kv_lists": (_i, [_vp, _i, _vp, _i, _i, _i, _d, _d, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "metok_debug_set": (_i, [_i, _i]),
    "metok_debug_build": (_i, []),
    "metok_status_string": (_c.c_char_p, [_i]),
    "metok_last_cuda_error": (_i, []),
    "metok_version": (_i, []),
}

_lib_handle = None


def exported_symbols() -> List[str]:
    return list(_SIGNATURES)


def lib():
    """Loads the CUDA library on first use; there is no other implementation."""
    global _lib_handle
    if _lib_handle is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2506_02850_b200.build` "
                "(the METok hot path has no CPU or PyTorch fallback)")
        h = _c.CDLL(LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(h, name)
            fn.restype = res
            fn.argtypes = args
        _lib_handle = h
    return _lib_handle


def _check(fn: str, status: int) -> None:
    if status != 0:
        L = lib()
        raise MetokError(fn, status, L.metok_status_string(status).decode(), L.metok_last_cuda_error())


def _dt(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else _vp(t.data_ptr())


def _stream() -> _vp:
    return _vp(torch.cuda.current_stream().cuda_stream)


def _cuda_contig(t: torch.Tensor, name: str) -> torch.Tensor:
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    return t


_ws_cache: Dict[tuple, torch.Tensor] = {}


def workspace(nbytes: int, device) -> torch.Tensor:
    """A reusable scratch buffer per device and stream: calls on one stream never overlap,
    calls on different streams may, so they must not share scratch."""
    key = (str(device), torch.cuda.current_stream(device).cuda_stream)
    buf = _ws_cache.get(key)
    if buf is None or buf.numel() < nbytes:
        buf = torch.empty(max(nbytes, 1 << 20), dtype=torch.uint8, device=device)
        _ws_cache[key] = buf
    return buf


# --------------------------------------------------------------------------- #


def metok_segment_events(feats: torch.Tensor, k: int, sim_mode: int = SIM_FLATTEN,
                         out: Optional[Dict[str, torch.Tensor]] = None) -> Dict[str, torch.Tensor]:
    """`out` (a dict returned by an earlier call with the same shapes) reuses its buffers."""
    feats = _cuda_contig(feats, "feats")
    T, N, d = feats.shape
    dev = feats.device
    L = lib()
    if out is not None:
        sims, boundaries, offsets, frame_event = out["_sims"], out["_boundaries"], out["_offsets"], out["frame_event"]
    else:
        sims = torch.empty(max(T - 1, 1), dtype=torch.float32, device=dev)
        boundaries = torch.empty(max(k - 1, 1), dtype=torch.int32, device=dev)
        offsets = torch.empty(max(k + 1, 2), dtype=torch.int32, device=dev)
        frame_event = torch.empty(T, dtype=torch.int32, device=dev)
    need = L.metok_segment_events_workspace_bytes(_dt(feats), T, N, d, sim_mode)
    ws = workspace(need, dev)
    st = L.metok_segment_events(_ptr(feats), _dt(feats), T, N, d, k, sim_mode, _ptr(sims), _ptr(boundaries),
                                _ptr(offsets), _ptr(frame_event), _ptr(ws), ws.numel(), _stream())
    _check("metok_segment_events", st)
    return {"sims": sims[: T - 1], "boundaries": boundaries[: max(k - 1, 0)], "event_offsets": offsets[: k + 1],
            "frame_event": frame_event, "_sims": sims, "_boundaries": boundaries, "_offsets": offsets}


def metok_segment_events_static(feats: torch.Tensor, k: int, sim_mode: int = SIM_FLATTEN) -> Dict[str, torch.Tensor]:
    """metok_segment_events for callers that must not allocate scratch: the library's
    built-in 1 MiB array is used instead of a workspace (problems that need more raise
    MetokError with status -6).  Calls on one device must not overlap on the GPU."""
    feats = _cuda_contig(feats, "feats")
    T, N, d = feats.shape
    dev = feats.device
    sims = torch.empty(max(T - 1, 1), dtype=torch.float32, device=dev)
    boundaries = torch.empty(max(k - 1, 1), dtype=torch.int32, device=dev)
    offsets = torch.empty(max(k + 1, 2), dtype=torch.int32, device=dev)
    frame_event = torch.empty(T, dtype=torch.int32, device=dev)
    st = lib().metok_segment_events_static(_ptr(feats), _dt(feats), T, N, d, k, sim_mode, _ptr(sims),
                                           _ptr(boundaries), _ptr(offsets), _ptr(frame_event), _stream())
    _check("metok_segment_events_static", st)
    return {"sims": sims[: T - 1], "boundaries": boundaries[: max(k - 1, 0)], "event_offsets": offsets[: k + 1],
            "frame_event": frame_event}


def metok_segment_score_events(feats: torch.Tensor, k: int, text_emb: torch.Tensor,
                               out: Optional[Dict[str, torch.Tensor]] = None) -> Dict[str, torch.Tensor]:
    """metok_segment_events (FLATTEN) plus the per-token text relevance and inverse norms of the
    same pass over `feats`; hand "token_score" / "token_inv_norm" on to metok_compress_vision."""
    feats = _cuda_contig(feats, "feats")
    text_emb = _cuda_contig(text_emb, "text_emb")
    T, N, d = feats.shape
    dev = feats.device
    L = lib()
    if out is None:
        out = {
            "_sims": torch.empty(max(T - 1, 1), dtype=torch.float32, device=dev),
            "_boundaries": torch.empty(max(k - 1, 1), dtype=torch.int32, device=dev),
            "_offsets": torch.empty(max(k + 1, 2), dtype=torch.int32, device=dev),
            "frame_event": torch.empty(T, dtype=torch.int32, device=dev),
            "token_score": torch.empty(T * N, dtype=torch.float32, device=dev),
            "token_inv_norm": torch.empty(T * N, dtype=torch.float32, device=dev),
        }
    need = L.metok_segment_score_events_workspace_bytes(_dt(feats), T, N, d)
    ws = workspace(need, dev)
    st = L.metok_segment_score_events(_ptr(feats), _dt(feats), T, N, d, k, _ptr(text_emb), _ptr(out["_sims"]),
                                      _ptr(out["_boundaries"]), _ptr(out["_offsets"]), _ptr(out["frame_event"]),
                                      _ptr(out["token_score"]), _ptr(out["token_inv_norm"]), _ptr(ws), ws.numel(),
                                      _stream())
    _check("metok_segment_score_events", st)
    out["sims"] = out["_sims"][: T - 1]
    out["boundaries"] = out["_boundaries"][: max(k - 1, 0)]
    out["event_offsets"] = out["_offsets"][: k + 1]
    return out


def vision_params(alpha: float, keep_key: float = 1.0, keep_nonkey: float = 1.0, event_agg: int = AGG_MEAN,
                  mode: int = MODE_TOPK_MERGE, beta: float = 0.5, s1: int = 2, s2: int = 3,
                  s1_nonkey: int = 4, s2_nonkey: int = 6) -> VisionParams:
    return VisionParams(alpha, event_agg, mode, keep_key, keep_nonkey, beta, s1, s2, s1_nonkey, s2_nonkey, None, None,
                        None)


def metok_compress_vision_bound(T: int, N: int, k: int, p: VisionParams) -> int:
    b = lib().metok_compress_vision_bound(T, N, k, _c.byref(p))
    if b < 0:
        _check("metok_compress_vision_bound", b)
    return b


def metok_compress_vision(feats: torch.Tensor, event_offsets: torch.Tensor, text_emb: torch.Tensor,
                          p: VisionParams, cap: Optional[int] = None,
                          out: Optional[Dict[str, torch.Tensor]] = None,
                          scored: Optional[Dict[str, torch.Tensor]] = None,
                          key_events: Optional[torch.Tensor] = None,
                          key_frames: Optional[torch.Tensor] = None) -> Dict[str, torch.Tensor]:
    """`scored` (the result of metok_segment_score_events on the same feats and text) makes the call
    skip its own scoring pass over `feats`; `key_events` (uint8 [k] on the device) replaces the
    call's own choice of key events, `key_frames` (uint8 [T], mode POOL) that of key frames."""
    feats = _cuda_contig(feats, "feats")
    event_offsets = _cuda_contig(event_offsets, "event_offsets")
    text_emb = _cuda_contig(text_emb, "text_emb")
    T, N, d = feats.shape
    k = event_offsets.numel() - 1
    dev = feats.device
    L = lib()
    if cap is None:
        cap = metok_compress_vision_bound(T, N, k, p)
    i32 = dict(dtype=torch.int32, device=dev)
    if out is not None:
        cap = out["out_src"].numel()
    else:
        out = {
            "out_feats": torch.empty((cap, d), dtype=feats.dtype, device=dev),
            "out_src": torch.empty(cap, **i32), "out_event": torch.empty(cap, **i32),
            "out_members": torch.empty(cap, **i32), "assign": torch.empty(T * N, **i32),
            "token_score": torch.empty(T * N, dtype=torch.float32, device=dev),
            "frame_score": torch.empty(T, dtype=torch.float32, device=dev),
            "event_score": torch.empty(k, dtype=torch.float32, device=dev),
            "event_is_key": torch.empty(k, dtype=torch.uint8, device=dev),
            "n_out": torch.zeros(1, **i32),
        }
    if scored is not None:
        out["token_score"] = scored["token_score"]
        p = VisionParams.from_buffer_copy(p)
        p.token_inv_norm = scored["token_inv_norm"].data_ptr()
    if key_events is not None:
        key_events = _cuda_contig(key_events, "key_events")
        if key_events.dtype != torch.uint8 or key_events.numel() != k:
            raise ValueError("key_events must be uint8 [k]")
        p = VisionParams.from_buffer_copy(p)
        p.key_events_given = key_events.data_ptr()
    if key_frames is not None:
        key_frames = _cuda_contig(key_frames, "key_frames")
        if key_frames.dtype != torch.uint8 or key_frames.numel() != T:
            raise ValueError("key_frames must be uint8 [T]")
        p = VisionParams.from_buffer_copy(p)
        p.key_frames_given = key_frames.data_ptr()
    need = L.metok_compress_vision_workspace_bytes(_dt(feats), T, N, d, k, cap, _c.byref(p))
    ws = workspace(need, dev)
    st = L.metok_compress_vision(_ptr(feats), _dt(feats), T, N, d, _ptr(event_offsets), k, _ptr(text_emb),
                                 _c.byref(p), _ptr(out["out_feats"]), _ptr(out["out_src"]), _ptr(out["out_event"]),
                                 _ptr(out["out_members"]), _ptr(out["assign"]), _ptr(out["token_score"]),
                                 _ptr(out["frame_score"]), _ptr(out["event_score"]), _ptr(out["event_is_key"]),
                                 _ptr(out["n_out"]), cap, _ptr(ws), ws.numel(), _stream())
    _check("metok_compress_vision", st)
    out["status"] = ws[:4].view(torch.int32)      # device status word (0, or -5 after a device-side timeout)
    return out


def metok_retention_budgets(alpha: float, r: float, stage: int, N0: Sequence[int]) -> List[int]:
    n0 = (_c.c_int32 * 2)(int(N0[0]), int(N0[1]))
    out = (_c.c_int32 * 2)()
    _check("metok_retention_budgets", lib().metok_retention_budgets(alpha, r, stage, n0, out))
    return [int(out[0]), int(out[1])]


def metok_prefill_prune(q_text: torch.Tensor, k_all: torch.Tensor, hidden: Optional[torch.Tensor], vis_start: int,
                        n_vis: int, token_group: torch.Tensor, group_budget: Sequence[int], softmax_scale: float,
                        out: Optional[Dict[str, torch.Tensor]] = None) -> Dict[str, torch.Tensor]:
    q_text = _cuda_contig(q_text, "q_text")
    k_all = _cuda_contig(k_all, "k_all")
    token_group = _cuda_contig(token_group, "token_group")
    Hq, Lt, dh = q_text.shape
    Hkv, S, _ = k_all.shape
    dev = q_text.device
    D = 0
    if hidden is not None:
        hidden = _cuda_contig(hidden, "hidden")
        D = hidden.shape[1]
    L = lib()
    G = len(group_budget)
    budgets = (_c.c_int32 * G)(*[int(b) for b in group_budget])
    if out is None:
        out = {
            "scores": torch.empty(n_vis, dtype=torch.float32, device=dev),
            "keep_idx": torch.empty(S, dtype=torch.int32, device=dev),
            "S_out": torch.zeros(1, dtype=torch.int32, device=dev),
            "hidden_out": None if hidden is None else torch.empty_like(hidden),
        }
    need = L.metok_prefill_prune_workspace_bytes(_dt(q_text), Hq, Hkv, Lt, S, dh, n_vis)
    ws = workspace(need, dev)
    st = L.metok_prefill_prune(_ptr(q_text), _ptr(k_all), _ptr(hidden), _dt(q_text), Hq, Hkv, Lt, S, dh, D, vis_start,
                               n_vis, _ptr(token_group), G, budgets, softmax_scale, _ptr(out["scores"]),
                               _ptr(out["keep_idx"]), _ptr(out["S_out"]), _ptr(out["hidden_out"]), _ptr(ws),
                               ws.numel(), _stream())
    _check("metok_prefill_prune", st)
    out["status"] = ws[:4].view(torch.int32)      # device status word (0, or -5 after a device-side timeout)
    return out


def metok_attention_scores(q_text: torch.Tensor, k_all: torch.Tensor, vis_start: int, n_vis: int,
                           softmax_scale: float, rows_total: int = 0,
                           scores: Optional[torch.Tensor] = None) -> torch.Tensor:
    """The scoring half of metok_prefill_prune for the heads given; `rows_total` = Hq * Lt over all
    ranks when the heads are sharded (the ranks' results then add up to the full score)."""
    q_text = _cuda_contig(q_text, "q_text")
    k_all = _cuda_contig(k_all, "k_all")
    Hq, Lt, dh = q_text.shape
    Hkv, S, _ = k_all.shape
    dev = q_text.device
    if scores is None:
        scores = torch.empty(n_vis, dtype=torch.float32, device=dev)
    L = lib()
    ws = workspace(L.metok_prefill_prune_workspace_bytes(_dt(q_text), Hq, Hkv, Lt, S, dh, n_vis), dev)
    st = L.metok_attention_scores(_ptr(q_text), _ptr(k_all), _dt(q_text), Hq, Hkv, Lt, S, dh, vis_start, n_vis,
                                  softmax_scale, rows_total, _ptr(scores), _ptr(ws), ws.numel(), _stream())
    _check("metok_attention_scores", st)
    return scores


def metok_prune_by_scores(scores: torch.Tensor, hidden: Optional[torch.Tensor], S: int, vis_start: int,
                          token_group: torch.Tensor, group_budget: Sequence[int],
                          dtype: Optional[torch.dtype] = None) -> Dict[str, torch.Tensor]:
    """The selection half of metok_prefill_prune on scores the caller holds."""
    scores = _cuda_contig(scores, "scores")
    token_group = _cuda_contig(token_group, "token_group")
    n_vis = scores.numel()
    dev = scores.device
    D = 0
    if hidden is not None:
        hidden = _cuda_contig(hidden, "hidden")
        D = hidden.shape[1]
        dtype = hidden.dtype
    code = F32 if dtype in (None, torch.float32) else BF16
    G = len(group_budget)
    budgets = (_c.c_int32 * G)(*[int(b) for b in group_budget])
    out = {"scores": scores, "keep_idx": torch.empty(S, dtype=torch.int32, device=dev),
           "S_out": torch.zeros(1, dtype=torch.int32, device=dev),
           "hidden_out": None if hidden is None else torch.empty_like(hidden)}
    L = lib()
    ws = workspace(L.metok_prune_by_scores_workspace_bytes(), dev)
    st = L.metok_prune_by_scores(_ptr(scores), _ptr(hidden), code, S, D, vis_start, n_vis, _ptr(token_group), G,
                                 budgets, _ptr(out["keep_idx"]), _ptr(out["S_out"]), _ptr(out["hidden_out"]), _ptr(ws),
                                 ws.numel(), _stream())
    _check("metok_prune_by_scores", st)
    out["status"] = ws[:4].view(torch.int32)
    return out


def head_shard(Hq: int, Hkv: int, rank: int, world: int):
    """Query heads [h0, h1) and KV heads [g0, g1) of `rank` when whole KV-head groups are dealt out."""
    if Hq % Hkv or Hkv % world:
        raise ValueError(f"{Hkv} KV heads (of {Hq} query heads) do not split over {world} ranks")
    per, rep = Hkv // world, Hq // Hkv
    return (rank * per * rep, (rank + 1) * per * rep), (rank * per, (rank + 1) * per)


def metok_prefill_prune_sharded(q_text_local: torch.Tensor, k_all_local: torch.Tensor, hidden: Optional[torch.Tensor],
                                vis_start: int, n_vis: int, token_group: torch.Tensor, group_budget: Sequence[int],
                                softmax_scale: float, group=None) -> Dict[str, torch.Tensor]:
    """One pruning level with the attention heads sharded over the ranks of `group` (head_shard): every
    rank scores with its own heads, one all-reduce (sum) of the n_vis scores, then every rank runs the
    same selection on the same scores."""
    import torch.distributed as dist
    world = dist.get_world_size(group) if dist.is_available() and dist.is_initialized() else 1
    Hq_local, Lt, _ = q_text_local.shape
    scores = metok_attention_scores(q_text_local, k_all_local, vis_start, n_vis, softmax_scale,
                                    rows_total=Hq_local * world * Lt)
    if world > 1:
        dist.all_reduce(scores, op=dist.ReduceOp.SUM, group=group)
    return metok_prune_by_scores(scores, hidden, k_all_local.shape[1], vis_start, token_group, group_budget,
                                 dtype=q_text_local.dtype)


def metok_prune_schedule_sizes(n_levels: int, alpha: float, r: float, N0: Sequence[int]) -> List[int]:
    n0 = (_c.c_int32 * 2)(int(N0[0]), int(N0[1]))
    out = (_c.c_int32 * (n_levels + 1))()
    _check("metok_prune_schedule_sizes", lib().metok_prune_schedule_sizes(n_levels, alpha, r, n0, out))
    return [int(v) for v in out]


def metok_prefill_prune_schedule(q_texts: Sequence[torch.Tensor], k_alls: Sequence[torch.Tensor],
                                 hiddens: Optional[Sequence[torch.Tensor]], vis_start: int, token_group: torch.Tensor,
                                 alpha: float, r: float, N0: Sequence[int],
                                 softmax_scale: float) -> List[Dict[str, torch.Tensor]]:
    """The pruning levels chained in one call: per level the tensors of that layer (rows of the
    survivors of the level before, in order).  Returns one dict per level."""
    n_levels = len(q_texts)
    token_group = _cuda_contig(token_group, "token_group")
    n_vis = token_group.numel()
    sizes = metok_prune_schedule_sizes(n_levels, alpha, r, N0)
    Hq, Lt, dh = q_texts[0].shape
    Hkv, S, _ = k_alls[0].shape
    dev = token_group.device
    D = 0 if hiddens is None else hiddens[0].shape[1]
    i32 = dict(dtype=torch.int32, device=dev)
    outs: List[Dict[str, torch.Tensor]] = []
    arr = (PruneLevel * n_levels)()
    for s in range(n_levels):
        q, k_ = _cuda_contig(q_texts[s], "q_text"), _cuda_contig(k_alls[s], "k_all")
        S_s = S - n_vis + sizes[s]
        if tuple(k_.shape) != (Hkv, S_s, dh):
            raise ValueError(f"level {s + 1}: k_all must be {(Hkv, S_s, dh)}, got {tuple(k_.shape)}")
        h = None if hiddens is None else _cuda_contig(hiddens[s], "hidden")
        o = {
            "scores": torch.empty(max(sizes[s], 1), dtype=torch.float32, device=dev),
            "keep_idx": torch.empty(S_s, **i32), "S_out": torch.zeros(1, **i32),
            "hidden_out": None if h is None else torch.empty_like(h),
            "token_group": token_group if s == 0 else torch.empty(max(sizes[s], 1), **i32),
            "origin": torch.empty(max(sizes[s], 1), **i32), "n_vis": sizes[s], "S": S_s,
        }
        arr[s] = PruneLevel(q.data_ptr(), k_.data_ptr(), None if h is None else h.data_ptr(),
                            None if h is None else o["hidden_out"].data_ptr(), o["scores"].data_ptr(),
                            o["keep_idx"].data_ptr(), o["S_out"].data_ptr(), o["token_group"].data_ptr(),
                            o["origin"].data_ptr())
        o["_inputs"] = (q, k_, h)                               # keep the tensors alive until the caller is done
        outs.append(o)
    n0 = (_c.c_int32 * 2)(int(N0[0]), int(N0[1]))
    L = lib()
    need = L.metok_prefill_prune_schedule_workspace_bytes(n_levels, _dt(q_texts[0]), Hq, Hkv, Lt, S, dh, n_vis, alpha, r, n0)
    if need == 0:
        _check("metok_prefill_prune_schedule", -1)
    ws = workspace(need, dev)
    status = torch.zeros(1, **i32)
    st = L.metok_prefill_prune_schedule(arr, n_levels, _dt(q_texts[0]), Hq, Hkv, Lt, S, dh, D, vis_start, n_vis, alpha, r,
                                        n0, softmax_scale, _ptr(status), _ptr(ws), ws.numel(), _stream())
    _check("metok_prefill_prune_schedule", st)
    for o in outs:
        o["status"] = status
        o["_schedule"] = (arr, n_levels, S, n_vis, alpha, r, n0)
    return outs


def metok_prune_schedule_kv_lists(levels: List[Dict[str, torch.Tensor]], level_layer: Sequence[int],
                                  L: int) -> Dict[str, object]:
    """K/V keep lists per layer from the keep lists recorded by metok_prefill_prune_schedule (its result is
    `levels`): {"keep_idx": int32 [L, S], "keep_len": int32 [L], "S_cur": list of L ints}."""
    arr, n_levels, S, n_vis, alpha, r, n0 = levels[0]["_schedule"]
    dev = levels[0]["keep_idx"].device
    keep_idx = torch.empty((L, S), dtype=torch.int32, device=dev)
    keep_len = torch.zeros(L, dtype=torch.int32, device=dev)
    s_cur = (_c.c_int32 * L)()
    layers = (_c.c_int32 * n_levels)(*[int(v) for v in level_layer])
    ws = workspace(4 * L, dev)
    st = lib().metok_prune_schedule_kv_lists(arr, n_levels, layers, L, S, n_vis, alpha, r, n0, _ptr(keep_idx), _ptr(keep_len),
                                             s_cur, _ptr(ws), ws.numel(), _stream())
    _check("metok_prune_schedule_kv_lists", st)
    return {"keep_idx": keep_idx, "keep_len": keep_len, "S_cur": [int(v) for v in s_cur]}


def metok_kv_compact(k_layers: Sequence[torch.Tensor], v_layers: Sequence[torch.Tensor], S_cur: int, policy: int,
                     vis_start: int, n_vis: int, l1: int = 0, keep_ratio: float = 1.0,
                     scores: Optional[torch.Tensor] = None, keep_idx: Optional[torch.Tensor] = None,
                     keep_len: Optional[torch.Tensor] = None,
                     new_len: Optional[torch.Tensor] = None) -> Dict[str, torch.Tensor]:
    nl = len(k_layers)
    for t in list(k_layers) + list(v_layers):
        _cuda_contig(t, "k/v layer")
    Hkv, S_cap, dh = k_layers[0].shape
    dev = k_layers[0].device
    L = lib()
    karr = (_vp * nl)(*[t.data_ptr() for t in k_layers])
    varr = (_vp * nl)(*[t.data_ptr() for t in v_layers])
    if keep_idx is None:
        keep_idx = torch.empty((nl, S_cur), dtype=torch.int32, device=dev)
        keep_len = torch.zeros(nl, dtype=torch.int32, device=dev)
    if new_len is None:
        new_len = torch.zeros(nl, dtype=torch.int32, device=dev)
    per_layer = 0
    if scores is not None:
        scores = _cuda_contig(scores, "scores")
        per_layer = 1 if scores.dim() == 2 else 0
    need = L.metok_kv_compact_workspace_bytes(_dt(k_layers[0]), nl, Hkv, S_cur, dh, policy, n_vis)
    ws = workspace(need, dev)
    st = L.metok_kv_compact(karr, varr, _dt(k_layers[0]), nl, Hkv, S_cap, S_cur, dh, policy, l1, keep_ratio,
                            vis_start, n_vis, _ptr(scores), per_layer, _ptr(keep_idx), _ptr(keep_len),
                            _ptr(new_len), _ptr(ws), ws.numel(), _stream())
    _check("metok_kv_compact", st)
    return {"keep_idx": keep_idx, "keep_len": keep_len, "new_len": new_len, "status": ws[:4].view(torch.int32)}


def metok_version() -> int:
    return lib().metok_version()


def metok_profile_begin() -> None:
    _check("metok_profile_begin", lib().metok_profile_begin())


def metok_profile_scope(label: Optional[str]) -> None:
    """Names the brackets recorded from now on: reported as "label/kernel"."""
    _check("metok_profile_scope", lib().metok_profile_scope(label.encode() if label else None))


def _profile(fn_name: str) -> Dict[str, Dict[str, float]]:
    buf = _c.create_string_buffer(1 << 16)
    n = getattr(lib(), fn_name)(buf, len(buf))
    if n < 0:
        _check(fn_name, n)
    out: Dict[str, Dict[str, float]] = {}
    for line in buf.value.decode().splitlines():
        name, cnt, ms = line.split()
        out[name] = {"launches": int(cnt), "ms": float(ms)}
    return out


def metok_profile_read() -> Dict[str, Dict[str, float]]:
    """Like metok_profile_end, but keeps the brackets: for replays of a graph that captured them."""
    return _profile("metok_profile_read")


def metok_profile_end() -> Dict[str, Dict[str, float]]:
    """{kernel name: {"launches": n, "ms": total}} for the launches since metok_profile_begin."""
    return _profile("metok_profile_end")

"""The debug library (lib/libmetok_debug.so): bounded waits that really run out, and range-checked indices.

A normal run never reaches the time-out and unwind code of the TMA / tcgen05 / bulk-copy pipelines.  In the
debug build a wait gives up after a few thousand polls and `metok_debug_set` makes the producer of one kernel
skip one copy: the consumer's wait runs out, the CTA unwinds (copies drained, tensor memory freed), the
kernel returns, the call's status word reads METOK_ERR_TIMEOUT, and the next ordinary call on the same GPU
gives the normal library's results bit for bit.  Nothing here faults, traps or leaves a kernel waiting.
The same build checks every data-dependent row and slot index against its range and counts the bad ones
(none may show up on the small and ragged cases)."""

import os

import numpy as np
import pytest
import torch

from paper_2506_02850_b200 import binding as B
from paper_2506_02850_b200 import build as builder
from paper_2506_02850_b200 import workloads as W

pytestmark = pytest.mark.gpu

TIMEOUT = -5
MERGE_ASSIGN, ATTN_STATS, ATTN_COLSUM, MERGE_AVG, GATHER_ROWS = 1, 2, 4, 8, 16


@pytest.fixture()
def debug_lib(monkeypatch):
    """binding.* calls go to the debug library inside the test; the normal one comes back afterwards."""
    assert os.path.exists(builder.DEBUG_LIB), "build it with `python -m paper_2506_02850_b200.build --debug`"
    normal = B.lib()
    assert normal.metok_debug_build() == 0 and normal.metok_debug_set(1, 1) == -2     # nothing to switch there
    monkeypatch.setattr(B, "_lib_handle", None)
    monkeypatch.setattr(B, "LIB_PATH", builder.DEBUG_LIB)
    dbg = B.lib()
    assert dbg.metok_debug_build() == 3
    yield dbg
    dbg.metok_debug_set(1, 0)
    torch.cuda.synchronize()


def _vision_case(seed=3, T=10, N=64, d=256):
    rng = np.random.default_rng(seed)
    offs = np.array([0, 3, 4, 10], dtype=np.int32)
    base = rng.standard_normal((3, N, d))
    V = np.concatenate([base[e][None] + 0.1 * rng.standard_normal((offs[e + 1] - offs[e], N, d)) for e in range(3)])
    t = rng.standard_normal(d)
    Vd = torch.from_numpy(V.astype(np.float32)).to(torch.bfloat16).cuda()
    td = torch.from_numpy(t.astype(np.float32)).to(torch.bfloat16).cuda()
    return Vd, torch.from_numpy(offs).cuda(), td, B.vision_params(0.5, 0.25, 0.25)


def _prefill_case(seed=4, Hq=4, Hkv=2, Lt=8, dh=64, n_vis=1500, D=256):
    rng = np.random.default_rng(seed)
    S = n_vis + Lt
    Q = torch.from_numpy(rng.standard_normal((Hq, Lt, dh)).astype(np.float32) * 0.3).to(torch.bfloat16).cuda()
    K = torch.from_numpy(rng.standard_normal((Hkv, S, dh)).astype(np.float32) * 0.3).to(torch.bfloat16).cuda()
    hidden = W.payload_torch(77, S, D, "bf16", "cuda")
    grp = torch.from_numpy((rng.random(n_vis) < 0.5).astype(np.int32)).cuda()
    return Q, K, hidden, 0, n_vis, grp, [300, 200], dh ** -0.5


def _vision_equal(a, b):
    n = int(a["n_out"].item())
    assert n == int(b["n_out"].item())
    for key in ("out_src", "out_event", "out_members"):
        assert torch.equal(a[key][:n], b[key][:n]), key
    assert torch.equal(a["assign"], b["assign"])
    assert torch.equal(a["out_feats"][:n].view(torch.int16), b["out_feats"][:n].view(torch.int16))


def _prefill_equal(a, b):
    n = int(a["S_out"].item())
    assert n == int(b["S_out"].item())
    assert torch.equal(a["scores"], b["scores"]) and torch.equal(a["keep_idx"][:n], b["keep_idx"][:n])
    assert torch.equal(a["hidden_out"][:n].view(torch.int16), b["hidden_out"][:n].view(torch.int16))


def test_wait_runs_out_in_the_stage1_kernels_and_the_next_call_is_clean(debug_lib):
    Vd, offs, td, p = _vision_case()
    want = {k_: (v.clone() if isinstance(v, torch.Tensor) else v) for k_, v in _normal_vision(Vd, offs, td, p).items()}
    for bit in (MERGE_ASSIGN, MERGE_AVG):
        assert debug_lib.metok_debug_set(1, bit) == 0
        got = B.metok_compress_vision(Vd, offs, td, p)
        torch.cuda.synchronize()                             # the kernels returned: nothing is left waiting
        assert int(got["status"].item()) == TIMEOUT, bit
        assert debug_lib.metok_debug_set(1, 0) == 0
        again = B.metok_compress_vision(Vd, offs, td, p)
        torch.cuda.synchronize()
        assert int(again["status"].item()) == 0
        _vision_equal(again, want)


def test_wait_runs_out_in_the_prefill_kernels_and_the_next_call_is_clean(debug_lib):
    args = _prefill_case()
    want = {k_: (v.clone() if isinstance(v, torch.Tensor) else v) for k_, v in _normal_prefill(args).items()}
    for bit in (ATTN_STATS, ATTN_COLSUM, GATHER_ROWS):
        assert debug_lib.metok_debug_set(1, bit) == 0
        got = B.metok_prefill_prune(*args)
        torch.cuda.synchronize()
        assert int(got["status"].item()) == TIMEOUT, bit
        assert debug_lib.metok_debug_set(1, 0) == 0
        again = B.metok_prefill_prune(*args)
        torch.cuda.synchronize()
        assert int(again["status"].item()) == 0
        _prefill_equal(again, want)


def _with_normal_library(fn):
    """fn() run against the normal library, whatever binding points to right now."""
    saved = (B._lib_handle, B.LIB_PATH)
    B._lib_handle, B.LIB_PATH = None, builder.LIB
    try:
        out = fn()
        torch.cuda.synchronize()
        return out
    finally:
        B._lib_handle, B.LIB_PATH = saved


def _normal_vision(Vd, offs, td, p):
    return _with_normal_library(lambda: B.metok_compress_vision(Vd, offs, td, p))


def _normal_prefill(args):
    return _with_normal_library(lambda: B.metok_prefill_prune(*args))


@pytest.mark.parametrize("case", ["tiny", "frames32", "ragged", "long_lists"])
def test_no_index_leaves_its_range(debug_lib, case):
    """Word 2 of the status area counts out-of-range row / slot indices met by the range-checked build."""
    if case == "ragged":
        Vd, offs, td, p = _vision_case(seed=9, T=7, N=37, d=72)
        offs = torch.tensor([0, 1, 2, 10], dtype=torch.int32).cuda()             # ten frames: events of 1, 1 and 8
    elif case == "long_lists":
        # 640 tokens and a handful of key tokens: member lists of a hundred and more, split into parts
        Vd, offs, td, _ = _vision_case(seed=12, T=10, N=64, d=136)
        p = B.vision_params(0.5, 0.006, 0.006)
    else:
        cfg = W.CONFIGS[case]
        vis = W.vision_inputs(cfg)
        tdt = torch.float32 if cfg.dtype == "f32" else torch.bfloat16
        Vd = torch.from_numpy(vis["V"]).to(tdt).cuda()
        td = torch.from_numpy(vis["t"]).to(tdt).cuda()
        offs = torch.from_numpy(np.asarray(vis["event_offsets"], dtype=np.int32)).cuda()
        p = B.vision_params(cfg.alpha, cfg.keep_enc, cfg.keep_enc)
    got = B.metok_compress_vision(Vd, offs, td, p)
    torch.cuda.synchronize()
    words = B.workspace(1, Vd.device)[:16].view(torch.int32)
    assert int(words[0].item()) == 0 and int(words[2].item()) == 0
    _vision_equal(got, _normal_vision(Vd, offs, td, p))
    args = _prefill_case(seed=11, n_vis=777 if case in ("ragged", "long_lists") else 1500)
    pf = B.metok_prefill_prune(*args)
    torch.cuda.synchronize()
    words = B.workspace(1, Vd.device)[:16].view(torch.int32)
    assert int(words[0].item()) == 0 and int(words[2].item()) == 0
    _prefill_equal(pf, _normal_prefill(args))

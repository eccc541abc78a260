"""The C-ABI library: loads, exports what include/metok.h declares, and its host-only
logic (validation, budgets, bounds, workspace sizes) behaves.  No GPU needed: every
call made here either is a pure host helper or fails validation before any launch."""

import ctypes
import os
import re

import pytest

from paper_2506_02850_b200 import binding as B
from paper_2506_02850_b200 import build as builder

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "metok.h")


@pytest.fixture(scope="module")
def lib():
    builder.build()
    return B.lib()


_real = {}


def device_pointers():
    """(pointer, pointer + 4, a second pointer) for arguments of calls that must be rejected before any
    launch.  Without a CUDA device they are made-up addresses (nothing can be launched anyway); with
    one they point into a real zero-filled 64 MiB allocation, so that a validation regression would
    launch on valid memory instead of a wild pointer."""
    try:
        import torch
        if torch.cuda.is_available():
            if "buf" not in _real:
                _real["buf"] = torch.zeros(1 << 26, dtype=torch.uint8, device="cuda")
            base = _real["buf"].data_ptr()
            return base, base + 4, base + (1 << 20)
    except Exception:
        pass
    return 0x10000, 0x10004, 0x20000


def declared_symbols():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(metok_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert len(names) >= 13
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(B.exported_symbols()) == names


def test_status_strings_and_version(lib):
    assert lib.metok_version() >= 100
    assert lib.metok_status_string(0) == b"ok"
    seen = {lib.metok_status_string(-i) for i in range(1, 6)}
    assert len(seen) == 5 and b"unknown status" not in seen
    assert lib.metok_status_string(-99) == b"unknown status"


def test_retention_budgets_follow_eq6_eq7(lib):
    # r = 0.55, alpha = 0.5 (LongVA setting): 1, r, r^2, 0 and 1, alpha*r, 0, 0
    assert B.metok_retention_budgets(0.5, 0.55, 0, (1000, 2000)) == [1000, 2000]
    assert B.metok_retention_budgets(0.5, 0.55, 1, (1000, 2000)) == [550, 550]
    assert B.metok_retention_budgets(0.5, 0.55, 2, (1000, 2000)) == [303, 0]
    assert B.metok_retention_budgets(0.5, 0.55, 3, (1000, 2000)) == [0, 0]
    assert B.metok_retention_budgets(0.5, 0.76, 2, (10000, 0)) == [5776, 0]
    for bad in [(0.0, 0.5, 1), (0.5, 1.5, 1), (0.5, 0.5, 4), (0.5, 0.5, -1)]:
        with pytest.raises(B.MetokError):
            B.metok_retention_budgets(bad[0], bad[1], bad[2], (1, 1))


def test_retention_budgets_match_oracle(lib):
    from oracle import metok_oracle as O
    for alpha, r in [(0.5, 0.55), (0.5, 0.76), (0.5, 0.65), (0.3, 0.9)]:
        for stage in range(4):
            for N0 in [(0, 0), (1, 1), (9216, 9216), (3333, 12345)]:
                assert B.metok_retention_budgets(alpha, r, stage, N0) == O.retention_budgets(alpha, r, stage, N0).tolist()


def test_compress_bound_and_workspace(lib):
    p = B.vision_params(0.5, 0.2, 0.2)
    assert B.metok_compress_vision_bound(128, 144, 16, p) == 3687 + 16      # ceil(.2*18432) + k
    assert B.metok_compress_vision_bound(8, 16, 2, B.vision_params(0.5, 1.0, 1.0)) == 128
    pool = B.vision_params(0.5, mode=B.MODE_POOL, beta=0.45, s1=2, s2=3, s1_nonkey=4, s2_nonkey=6)
    assert B.metok_compress_vision_bound(128, 144, 16, pool) == 128 * 36
    with pytest.raises(B.MetokError):
        B.metok_compress_vision_bound(128, 143, 16, pool)                    # N is not a square
    with pytest.raises(B.MetokError):
        B.metok_compress_vision_bound(4, 16, 5, p)                           # k > T
    for fn, args in [("metok_segment_events_workspace_bytes", (B.BF16, 128, 144, 3584, 0)),
                     ("metok_prefill_prune_workspace_bytes", (B.BF16, 28, 4, 64, 18496, 128, 18432)),
                     ("metok_kv_compact_workspace_bytes", (B.BF16, 28, 4, 18496, 128, 1, 18432))]:
        n = getattr(lib, fn)(*args)
        assert 0 < n < (1 << 30) and n % 256 == 0
    n = lib.metok_compress_vision_workspace_bytes(B.BF16, 128, 144, 3584, 16, 3703, ctypes.byref(p))
    assert 0 < n < (1 << 30)


def test_validation_rejects_before_any_launch(lib):
    """Bad arguments return INVALID_ARG / UNSUPPORTED / WORKSPACE without touching the GPU
    (see device_pointers for what the non-null pointers are)."""
    p0, p_odd, p1 = device_pointers()
    fake = ctypes.c_void_p(p0)
    odd = ctypes.c_void_p(p_odd)
    null = ctypes.c_void_p(0)
    seg = lib.metok_segment_events
    ok_args = [fake, B.BF16, 8, 16, 64, 2, 0, fake, fake, fake, fake, fake, 1 << 20, null]

    def call(**kw):
        a = list(ok_args)
        names = ["feats", "dtype", "T", "N", "d", "k", "sim_mode", "sims", "boundaries", "event_offsets",
                 "frame_event", "ws", "ws_bytes", "stream"]
        for k_, v in kw.items():
            a[names.index(k_)] = v
        return seg(*a)

    assert call(feats=null) == -1
    assert call(feats=odd) == -1
    assert call(k=0) == -1 and call(k=9) == -1
    assert call(T=0) == -1 and call(d=0) == -1 and call(dtype=7) == -1 and call(sim_mode=3) == -1
    assert call(d=12) == -2                                   # 24-byte rows
    assert call(T=10000, k=2) == -2
    assert call(ws=null) == -3 and call(ws_bytes=0) == -3

    p = B.vision_params(0.5, 0.5, 0.5)
    cv = lib.metok_compress_vision
    base = [fake, B.BF16, 8, 16, 64, fake, 2, fake, ctypes.byref(p)] + [fake] * 10 + [128, fake, 1 << 24, null]
    bad_alpha = B.vision_params(1.5, 0.5, 0.5)
    b2 = list(base); b2[8] = ctypes.byref(bad_alpha)
    assert cv(*b2) == -1
    b3 = list(base); b3[19] = 3                               # cap below the bound
    assert cv(*b3) == -1
    b4 = list(base); b4[0] = null
    assert cv(*b4) == -1
    b5 = list(base); b5[21] = 0                               # workspace too small
    assert cv(*b5) == -3

    pp = lib.metok_prefill_prune
    budgets = (ctypes.c_int32 * 2)(3, 3)
    pbase = [fake, fake, fake, B.BF16, 28, 4, 16, 160, 128, 3584, 0, 144, fake, 2, budgets, 0.088,
             fake, fake, fake, fake, fake, 1 << 26, null]
    def pcall(idx, val):
        a = list(pbase); a[idx] = val
        return pp(*a)
    assert pcall(4, 27) == -1                                 # Hq % Hkv
    assert pcall(6, 200) == -1                                # Lt > S
    assert pcall(11, 150) == -1                               # visual span overlaps the text queries
    assert pcall(13, 0) == -1 and pcall(13, 65) == -1         # G
    assert pcall(8, 96) == -2                                 # head dim
    assert pcall(9, 100) == -2                                # 200-byte hidden rows
    assert pcall(21, 16) == -3
    neg = (ctypes.c_int32 * 2)(3, -1)
    assert pcall(14, neg) == -1

    kv = lib.metok_kv_compact
    ptrs = (ctypes.c_void_p * 2)(p0, p1)
    kbase = [ptrs, ptrs, B.BF16, 2, 4, 160, 160, 128, B.KV_TOPK, 0, 0.1, 0, 144, fake, 0, fake, fake, fake,
             fake, 1 << 20, null]
    def kcall(idx, val):
        a = list(kbase); a[idx] = val
        return kv(*a)
    assert kcall(6, 161) == -1                                # S_cur > S_cap
    assert kcall(8, 5) == -1                                  # policy
    assert kcall(10, 1.5) == -1                               # ratio
    assert kcall(12, 200) == -1                               # span beyond S_cur
    assert kcall(13, null) == -1                              # TOPK needs scores
    assert kcall(7, 100) == -2                                # 200-byte rows
    assert kcall(18, null) == -3
    badptrs = (ctypes.c_void_p * 2)(p0, 0)
    assert kcall(0, badptrs) == -1


def test_missing_library_fails_loudly(tmp_path, monkeypatch):
    monkeypatch.setattr(B, "_lib_handle", None)
    monkeypatch.setattr(B, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        B.lib()


def test_prune_schedule_sizes_and_validation(lib):
    """Sizes of the levels follow Eq. 6/7 on the host; bad schedules are rejected before any launch."""
    assert B.metok_prune_schedule_sizes(3, 0.5, 0.55, (200, 100)) == [300, 110 + 28, 61, 0]
    from oracle import metok_oracle as O
    for alpha, r, N0 in [(0.5, 0.76, (3000, 3272)), (0.5, 0.65, (1, 1)), (0.3, 0.9, (7, 0))]:
        want = [int(O.retention_budgets(alpha, r, s, N0).sum()) for s in range(4)]
        assert B.metok_prune_schedule_sizes(3, alpha, r, N0) == want
    with pytest.raises(B.MetokError):
        B.metok_prune_schedule_sizes(4, 0.5, 0.5, (1, 1))
    p0 = device_pointers()[0]
    fake, null = ctypes.c_void_p(p0), ctypes.c_void_p(0)
    lv = (B.PruneLevel * 3)()
    for s in range(3):
        lv[s] = B.PruneLevel(*([p0] * 9))
    n0 = (ctypes.c_int32 * 2)(200, 100)
    fn = lib.metok_prefill_prune_schedule
    args = [lv, 3, B.BF16, 28, 4, 16, 316, 128, 3584, 0, 300, 0.5, 0.55, n0, 0.088, fake, fake, 1 << 26, null]

    def call(idx, val):
        a = list(args); a[idx] = val
        return fn(*a)
    assert call(1, 0) == -1 and call(1, 4) == -1              # number of levels
    assert call(10, 299) == -1                                # N0 does not sum to n_vis
    assert call(12, 1.5) == -1                                # r
    assert call(15, null) == -1                               # status pointer
    n0_empty = (ctypes.c_int32 * 2)(0, 300)                   # no key-event tokens: level 3 would get no visual token
    assert call(13, n0_empty) == -1
    assert lib.metok_prefill_prune_schedule_workspace_bytes(3, B.BF16, 28, 4, 16, 316, 128, 300, 0.5, 0.55, n0) > 0
    assert lib.metok_prefill_prune_schedule_workspace_bytes(3, B.BF16, 28, 4, 16, 316, 128, 299, 0.5, 0.55, n0) == 0


def test_prune_schedule_checks_every_level_before_the_first_launch(lib):
    """A bad argument at a later level (null q_text at level 2, a misaligned K at level 3, a workspace
    too small for the largest level) is rejected with nothing launched: the library's own launch
    counter stays at zero."""
    p0, p_odd, _ = device_pointers()
    null = ctypes.c_void_p(0)
    n0 = (ctypes.c_int32 * 2)(200, 100)
    fn = lib.metok_prefill_prune_schedule
    names = [f[0] for f in B.PruneLevel._fields_]

    def levels(**bad):
        lv = (B.PruneLevel * 3)()
        for s in range(3):
            lv[s] = B.PruneLevel(*([p0] * 9))
        for key, (s, val) in bad.items():
            assert key in names
            setattr(lv[s], key, val)
        return lv

    def call(lv, ws_bytes=1 << 26):
        assert lib.metok_profile_begin() == 0
        rc = fn(lv, 3, B.BF16, 28, 4, 16, 316, 128, 3584, 0, 300, 0.5, 0.55, n0, 0.088, ctypes.c_void_p(p0),
                ctypes.c_void_p(p0), ws_bytes, null)
        launched = lib.metok_profile_end(None, 0)
        return rc, launched

    assert call(levels(q_text=(1, None))) == (-1, 0)
    assert call(levels(k_all=(2, p_odd))) == (-1, 0)
    assert call(levels(keep_idx=(1, None))) == (-1, 0)
    assert call(levels(hidden_out=(2, None))) == (-1, 0)      # hidden without hidden_out
    assert call(levels(), ws_bytes=4096) == (-3, 0)

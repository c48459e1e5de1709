"""GPU parity of swaa_decode (through the C ABI) against the float64 oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_2512_10411_b200 as swaa
from paper_2512_10411_b200 import inputs
from helpers import check_against_oracle

pytestmark = pytest.mark.gpu


def _run_decode(q, kc, vc, seqlens, W, S, full, scale=0.0, poison=True):
    B, Hq, D = q.shape
    _, Lmax, Hkv, _ = kc.shape
    nbytes = swaa.decode_workspace_size(B, Hq, Hkv, D, Lmax, W, S, full)
    # guard bands around output and workspace catch out-of-bounds stores
    guard = 4096
    ws_all = torch.full((nbytes + 2 * guard,), 0xA5, dtype=torch.uint8, device="cuda")
    ws = ws_all[guard:guard + nbytes]
    assert ws.data_ptr() % 256 == 0
    out_all = torch.full((B * Hq * D + 2 * 1024,), float("nan"), dtype=torch.bfloat16, device="cuda")
    out = out_all[1024:1024 + B * Hq * D].view(B, Hq, D)
    swaa.swaa_decode(q, kc, vc, out, seqlens, W, S, full, ws, scale=scale)
    status = swaa.last_device_status()
    assert torch.isnan(out_all[:1024]).all() and torch.isnan(out_all[-1024:]).all(), "store outside `out`"
    assert (ws_all[:guard] == 0xA5).all() and (ws_all[-guard:] == 0xA5).all(), "store outside the workspace"
    return out, status


SHAPES = [
    # B, Lmax, Hq, Hkv, D, seqlens
    (3, 300, 4, 2, 64, (300, 1, 17)),
    (2, 515, 8, 1, 128, (515, 130)),
    (2, 200, 16, 1, 128, (200, 33)),     # G = 16: two 8-head blocks
    (1, 260, 32, 1, 64, (259,)),         # G = 32: two head chunks per kv head
    (2, 257, 6, 2, 128, (16, 257)),      # G = 3: padded heads
    (1, 9000, 8, 2, 128, (8999,)),       # several key splits
    (4, 20000, 32, 8, 128, (20000, 4101, 4100, 1)),
]
POLICIES = [(1, 0, True), (1, 0, False), (16, 0, False), (128, 4, False), (4096, 4, False), (100, 300, False),
            (7, 3, False)]


@pytest.mark.parametrize("shape", SHAPES)
def test_decode_matches_oracle(shape):
    B, Lmax, Hq, Hkv, D, sl = shape
    cfg = inputs.DecodeConfig("t", B, Lmax, Hq, Hkv, D, 0, 0, seed=100 + Lmax, seqlens=sl)
    q, kc, vc, seqlens = inputs.make_decode_inputs(cfg, "cuda")
    qh, kh, vh = inputs.to_f32_numpy(q), inputs.to_f32_numpy(kc), inputs.to_f32_numpy(vc)
    for W, S, full in POLICIES:
        out, status = _run_decode(q, kc, vc, seqlens, W, S, full)
        assert status == 0
        ref = oracle.decode(qh, kh, vh, sl, W, S, full)
        check_against_oracle(out, ref["out"], f"decode {shape} W={W} S={S} full={full}")


def test_decode_window_one_returns_own_value_exactly():
    cfg = inputs.DecodeConfig("t", 3, 1000, 8, 2, 128, 0, 0, seed=7, seqlens=(1000, 5, 333))
    q, kc, vc, seqlens = inputs.make_decode_inputs(cfg, "cuda")
    out, status = _run_decode(q, kc, vc, seqlens, 1, 0, False)
    assert status == 0
    for b, n in enumerate(cfg.seqlens):
        want = vc[b, n - 1].repeat_interleave(4, dim=0)
        assert torch.equal(out[b], want)


def test_decode_visible_set_is_bit_exact():
    """Q = 0 and one-hot V: out[c] > 0 exactly where key t*D+c is visible, exactly 0 elsewhere."""
    B, Lmax, Hq, Hkv, D = 2, 1024, 4, 2, 64
    sl = (1024, 700)
    q = torch.zeros((B, Hq, D), dtype=torch.bfloat16, device="cuda")
    kc = torch.randn((B, Lmax, Hkv, D), device="cuda").to(torch.bfloat16)
    seqlens = torch.tensor(sl, dtype=torch.int32, device="cuda")
    for W, S, full in ((100, 3, False), (1, 0, False), (64, 70, False), (5, 0, True)):
        seen = np.zeros((B, Lmax), dtype=bool)
        for t in range(Lmax // D):
            vc = torch.zeros((B, Lmax, Hkv, D), dtype=torch.bfloat16, device="cuda")
            idx = torch.arange(D, device="cuda")
            vc[:, t * D + idx, :, idx] = 1.0
            out, status = _run_decode(q, kc, vc, seqlens, W, S, full)
            assert status == 0
            o = out.float().cpu().numpy()
            assert (o >= 0).all()
            for h in range(Hq):
                assert np.array_equal(o[:, h] > 0, o[:, 0] > 0)
            seen[:, t * D:(t + 1) * D] = o[:, 0] > 0
        for b, n in enumerate(sl):
            want = np.array([oracle.visible(n - 1, j, W, S, full) for j in range(Lmax)])
            assert np.array_equal(seen[b], want), (W, S, full, b)


def test_decode_never_uses_cache_entries_past_seqlens():
    """Entries past seqlens[b] hold NaN: they share 64-entry tiles with visible entries and must not leak."""
    cfg = inputs.DecodeConfig("t", 3, 700, 8, 2, 128, 0, 0, seed=21, seqlens=(650, 3, 129))
    q, kc, vc, seqlens = inputs.make_decode_inputs(cfg, "cuda")
    for b, n in enumerate(cfg.seqlens):
        kc[b, n:] = float("nan")
        vc[b, n:] = float("nan")
    qh, kh, vh = inputs.to_f32_numpy(q), inputs.to_f32_numpy(kc), inputs.to_f32_numpy(vc)
    for W, S, full in ((1, 0, True), (100, 4, False), (64, 0, False), (1, 0, False)):
        out, status = _run_decode(q, kc, vc, seqlens, W, S, full)
        assert status == 0
        ref = oracle.decode(qh, kh, vh, cfg.seqlens, W, S, full)
        check_against_oracle(out, ref["out"], f"NaN tail W={W} S={S} full={full}")


@pytest.mark.parametrize("D", [64, 128])
def test_decode_many_short_sequences(D):
    """More sequences than threads in a block, random lengths: many whole items per block, few cut ones."""
    rng = np.random.default_rng(33)
    B, Lmax = 437, 260
    sl = tuple(int(x) for x in rng.integers(1, Lmax + 1, B))
    cfg = inputs.DecodeConfig("t", B, Lmax, 8, 2, D, 0, 0, seed=34, seqlens=sl)
    q, kc, vc, seqlens = inputs.make_decode_inputs(cfg, "cuda")
    qh, kh, vh = inputs.to_f32_numpy(q), inputs.to_f32_numpy(kc), inputs.to_f32_numpy(vc)
    for W, S, full in ((1, 0, True), (70, 5, False), (128, 100, False)):
        out, status = _run_decode(q, kc, vc, seqlens, W, S, full)
        assert status == 0
        ref = oracle.decode(qh, kh, vh, sl, W, S, full)
        check_against_oracle(out, ref["out"], f"many sequences D={D} W={W} S={S} full={full}")


def test_decode_reports_bad_seqlens_and_zero_fills():
    cfg = inputs.DecodeConfig("t", 3, 128, 4, 2, 64, 0, 0, seed=9, seqlens=(128, 0, 129))
    q, kc, vc, seqlens = inputs.make_decode_inputs(cfg, "cuda")
    out, status = _run_decode(q, kc, vc, seqlens, 16, 0, False)
    assert status == -5
    assert swaa.last_device_status() == 0  # reading clears it
    assert (out[1] == 0).all() and (out[2] == 0).all()
    ref = oracle.decode(inputs.to_f32_numpy(q[:1]), inputs.to_f32_numpy(kc[:1]), inputs.to_f32_numpy(vc[:1]),
                        [128], 16, 0, False)
    check_against_oracle(out[:1], ref["out"], "valid sequence next to bad ones")


def test_decode_argument_errors():
    cfg = inputs.DecodeConfig("t", 1, 64, 4, 2, 64, 0, 0, seed=1)
    q, kc, vc, seqlens = inputs.make_decode_inputs(cfg, "cuda")
    out = torch.empty_like(q)
    ws = torch.empty(1 << 20, dtype=torch.uint8, device="cuda")
    with pytest.raises(swaa.SwaaError) as e:
        swaa.swaa_decode(q, kc, vc, out, seqlens, 0, 0, False, ws)
    assert e.value.status == -1
    with pytest.raises(swaa.SwaaError) as e:
        swaa.swaa_decode(q, kc, vc, out, seqlens, 8, 0, False, ws[:16])
    assert e.value.status == -4
    q3 = torch.empty((1, 3, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(swaa.SwaaError) as e:
        swaa.swaa_decode(q3, kc, vc, torch.empty_like(q3), seqlens, 8, 0, False, ws)
    assert e.value.status == -2


@pytest.mark.parametrize("full", [True, False])
def test_decode_full_size_workload(full):
    """Workload 4 at full size (B=16, 65536-entry cache, Hq=32, Hkv=8, D=128), every output row."""
    cfg = inputs.cfg_decode()
    q, kc, vc, seqlens = inputs.make_decode_inputs(cfg, "cuda")
    out, status = _run_decode(q, kc, vc, seqlens, cfg.window, cfg.n_sink, full)
    assert status == 0
    qh = inputs.to_f32_numpy(q)
    worst = (0.0, 0.0)
    for b in range(0, cfg.B, 4):  # host copies of four sequences at a time keep memory modest
        kh, vh = inputs.to_f32_numpy(kc[b:b + 4]), inputs.to_f32_numpy(vc[b:b + 4])
        ref = oracle.decode(qh[b:b + 4], kh, vh, [cfg.Lmax] * 4, cfg.window, cfg.n_sink, full)
        assert (ref["nvis"] == (cfg.Lmax if full else cfg.window + cfg.n_sink)).all()
        r = check_against_oracle(out[b:b + 4], ref["out"], f"cfg4 full={full} b={b}")
        worst = max(worst, r)
    print(f"cfg4 decode full={full}: max abs err {worst[0]:.3e}, max rel err {worst[1]:.3e}")


def test_decode_on_a_trimmed_ring_cache_equals_swa_decode():
    """A pure-SWA layer keeps n_sink + window cache entries (ring); full attention over them is the SWA decode."""
    B, Hq, Hkv, D, W, S = 3, 8, 2, 128, 200, 5
    sl = (1000, 150, 206)
    cfg = inputs.DecodeConfig("t", B, 1000, Hq, Hkv, D, W, S, seed=55, seqlens=sl)
    q, kc, vc, seqlens = inputs.make_decode_inputs(cfg, "cuda")
    cap = S + W
    kt = torch.full((B, cap, Hkv, D), float("nan"), dtype=torch.bfloat16, device="cuda")
    vt = torch.full_like(kt, float("nan"))
    for b, n in enumerate(sl):
        for pos in range(n):  # the order in which a serving loop would append
            slot = swaa.trimmed_cache_slot(pos, W, S)
            kt[b, slot] = kc[b, pos]
            vt[b, slot] = vc[b, pos]
    tl = torch.tensor([swaa.trimmed_cache_len(n, W, S) for n in sl], dtype=torch.int32, device="cuda")
    out, status = _run_decode(q, kt, vt, tl, 1, 0, True)
    assert status == 0
    ref = oracle.decode(inputs.to_f32_numpy(q), inputs.to_f32_numpy(kc), inputs.to_f32_numpy(vc), sl, W, S, False)
    check_against_oracle(out, ref["out"], "trimmed ring cache")

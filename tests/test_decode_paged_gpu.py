"""GPU parity of swaa_decode_paged (through the C ABI) against the float64 oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_2512_10411_b200 as swaa
from paper_2512_10411_b200 import inputs
from helpers import check_against_oracle

pytestmark = pytest.mark.gpu


def make_paged(B, Hq, Hkv, D, page, sl, seed, spare_pages=7, poison=True):
    """Random q and a paged cache: pages handed out in random order, unused pages and the rows past each
    sequence's last entry hold NaN.  Returns device tensors and the block table."""
    g = torch.Generator(device="cuda").manual_seed(seed)
    rng = np.random.default_rng(seed)
    blocks = [(n + page - 1) // page for n in sl]
    max_blocks = max(blocks) + 1
    num_pages = sum(blocks) + spare_pages
    q = torch.randn((B, Hq, D), generator=g, device="cuda").to(torch.bfloat16)
    kp = torch.randn((num_pages, page, Hkv, D), generator=g, device="cuda").to(torch.bfloat16)
    vp = torch.randn((num_pages, page, Hkv, D), generator=g, device="cuda").to(torch.bfloat16)
    perm = rng.permutation(num_pages)
    bt = np.full((B, max_blocks), -1, dtype=np.int32)
    used = np.zeros((num_pages, page), dtype=bool)
    nxt = 0
    for b in range(B):
        for blk in range(blocks[b]):
            pg = int(perm[nxt]); nxt += 1
            bt[b, blk] = pg
            used[pg, :min(page, sl[b] - blk * page)] = True
    if poison:
        mask = torch.as_tensor(~used, device="cuda")
        kp[mask] = float("nan")
        vp[mask] = float("nan")
    return q, kp, vp, torch.as_tensor(bt, device="cuda"), torch.tensor(sl, dtype=torch.int32, device="cuda")


def run_paged(q, kp, vp, bt, seqlens, W, S, full, scale=0.0):
    B, Hq, D = q.shape
    _, page, Hkv, _ = kp.shape
    nbytes = swaa.decode_paged_workspace_size(B, Hq, Hkv, D, bt.shape[1], page, W, S, full)
    guard = 4096
    ws_all = torch.full((nbytes + 2 * guard,), 0xA5, dtype=torch.uint8, device="cuda")
    ws = ws_all[guard:guard + nbytes]
    out_all = torch.full((B * Hq * D + 2 * 1024,), float("nan"), dtype=torch.bfloat16, device="cuda")
    out = out_all[1024:1024 + B * Hq * D].view(B, Hq, D)
    swaa.swaa_decode_paged(q, kp, vp, out, bt, seqlens, W, S, full, ws, scale=scale)
    status = swaa.last_device_status()
    assert torch.isnan(out_all[:1024]).all() and torch.isnan(out_all[-1024:]).all(), "store outside `out`"
    assert (ws_all[:guard] == 0xA5).all() and (ws_all[-guard:] == 0xA5).all(), "store outside the workspace"
    return out, status


SHAPES = [
    # B, Hq, Hkv, D, page_size, seqlens
    (3, 4, 2, 64, 64, (300, 1, 17)),
    (2, 8, 1, 128, 128, (515, 130)),
    (2, 16, 1, 128, 64, (200, 33)),          # G = 16: two 8-head blocks
    (2, 6, 2, 128, 256, (16, 257)),          # G = 3: padded heads
    (1, 8, 2, 128, 64, (8999,)),             # cut over several blocks
    (4, 32, 8, 128, 128, (20000, 4101, 4100, 1)),
]
POLICIES = [(1, 0, True), (1, 0, False), (16, 0, False), (128, 4, False), (4096, 4, False), (100, 300, False),
            (7, 3, False), (65, 64, False), (200, 70, False)]


@pytest.mark.parametrize("shape", SHAPES)
def test_paged_decode_matches_oracle(shape):
    B, Hq, Hkv, D, page, sl = shape
    q, kp, vp, bt, seqlens = make_paged(B, Hq, Hkv, D, page, sl, seed=600 + sum(sl))
    qh, kh, vh = inputs.to_f32_numpy(q), inputs.to_f32_numpy(kp), inputs.to_f32_numpy(vp)
    for W, S, full in POLICIES:
        out, status = run_paged(q, kp, vp, bt, seqlens, W, S, full)
        assert status == 0
        ref = oracle.decode_paged(qh, kh, vh, bt.cpu().numpy(), sl, W, S, full)
        check_against_oracle(out, ref["out"], f"paged decode {shape} W={W} S={S} full={full}")


def test_paged_decode_visible_set_is_bit_exact():
    """Q = 0 and one-hot V (in logical entry order): out[c] > 0 exactly where entry t*D+c is visible."""
    B, Hq, Hkv, D, page = 2, 4, 2, 64, 64
    sl = (1000, 700)
    q, kp, vp, bt, seqlens = make_paged(B, Hq, Hkv, D, page, sl, seed=5, poison=False)
    q.zero_()
    btn = bt.cpu().numpy()
    Lp = 1024
    for W, S, full in ((100, 3, False), (1, 0, False), (64, 70, False), (130, 0, False), (5, 0, True)):
        seen = np.zeros((B, Lp), dtype=bool)
        for t in range(Lp // D):
            vp.zero_()
            for b in range(B):
                for c in range(D):
                    j = t * D + c
                    if j < sl[b]:
                        vp[int(btn[b, j // page]), j % page, :, c] = 1.0
            out, status = run_paged(q, kp, vp, bt, seqlens, W, S, full)
            assert status == 0
            o = out.float().cpu().numpy()
            assert (o >= 0).all()
            seen[:, t * D:(t + 1) * D] = o[:, 0] > 0
        for b, n in enumerate(sl):
            want = np.array([j < n and oracle.visible(n - 1, j, W, S, full) for j in range(Lp)])
            assert np.array_equal(seen[b], want), (W, S, full, b)


def test_paged_decode_reports_a_bad_page_index():
    q, kp, vp, bt, seqlens = make_paged(2, 4, 2, 64, 64, (100, 64), seed=9, poison=False)
    bt2 = bt.clone()
    bt2[0, 1] = kp.shape[0] + 5
    out, status = run_paged(q, kp, vp, bt2, seqlens, 1, 0, True)
    assert status == -5
    assert swaa.last_device_status() == 0
    ref = oracle.decode_paged(inputs.to_f32_numpy(q[1:]), inputs.to_f32_numpy(kp), inputs.to_f32_numpy(vp),
                              bt.cpu().numpy()[1:], [64], 1, 0, True)
    check_against_oracle(out[1:], ref["out"], "sequence next to the one with the bad page")


def test_paged_decode_argument_errors():
    q, kp, vp, bt, seqlens = make_paged(1, 4, 2, 64, 64, (64,), seed=1, poison=False)
    ws = torch.empty(1 << 20, dtype=torch.uint8, device="cuda")
    kp96 = torch.zeros((4, 96, 2, 64), dtype=torch.bfloat16, device="cuda")  # page size not a multiple of 64
    with pytest.raises(swaa.SwaaError) as e:
        swaa.swaa_decode_paged(q, kp96, kp96, torch.empty_like(q), bt, seqlens, 8, 0, False, ws)
    assert e.value.status == -2
    with pytest.raises(swaa.SwaaError) as e:
        swaa.swaa_decode_paged(q, kp, vp, torch.empty_like(q), bt, seqlens, 8, 0, False, ws[:16])
    assert e.value.status == -4


@pytest.mark.parametrize("full", [True, False])
def test_paged_decode_full_size_workload(full):
    """Workload 4 at full size with 256-entry pages in random order (B=16, 65536 entries each), every row."""
    cfg = inputs.cfg_decode()
    sl = (cfg.Lmax,) * cfg.B
    q, kp, vp, bt, seqlens = make_paged(cfg.B, cfg.Hq, cfg.Hkv, cfg.D, 256, sl, seed=44, spare_pages=3, poison=False)
    out, status = run_paged(q, kp, vp, bt, seqlens, cfg.window, cfg.n_sink, full)
    assert status == 0
    qh, btn = inputs.to_f32_numpy(q), bt.cpu().numpy()
    for b in range(0, cfg.B, 4):  # four sequences at a time keep the host copies modest
        pages = np.unique(btn[b:b + 4, :cfg.Lmax // 256])
        remap = np.zeros(kp.shape[0], dtype=np.int64)
        remap[pages] = np.arange(pages.shape[0])
        idx = torch.as_tensor(pages, device="cuda")
        ref = oracle.decode_paged(qh[b:b + 4], inputs.to_f32_numpy(kp[idx]), inputs.to_f32_numpy(vp[idx]),
                                  remap[btn[b:b + 4, :cfg.Lmax // 256]], sl[b:b + 4], cfg.window, cfg.n_sink, full)
        check_against_oracle(out[b:b + 4], ref["out"], f"paged cfg4 full={full} b={b}")

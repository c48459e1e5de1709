"""GPU parity of swaa_prefill_paged (through the C ABI) against the float64 oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_2512_10411_b200 as swaa
from paper_2512_10411_b200 import inputs
from helpers import check_against_oracle

pytestmark = pytest.mark.gpu

GUARD = 4096


def make_paged(lq, lk, Hq, Hkv, D, page, seed, spare_pages=3, poison=True):
    """Random queries and a paged K/V pool: pages handed out in random order; unused pages and the rows past
    each sequence's last key hold NaN."""
    g = torch.Generator(device="cuda").manual_seed(seed)
    rng = np.random.default_rng(seed)
    B = len(lq)
    blocks = [(n + page - 1) // page for n in lk]
    max_blocks = max(blocks) + 1
    num_pages = sum(blocks) + spare_pages
    q = torch.randn((sum(lq), Hq, D), generator=g, device="cuda").to(torch.bfloat16)
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
            used[pg, :min(page, lk[b] - blk * page)] = True
    if poison:
        mask = torch.as_tensor(~used, device="cuda")
        kp[mask] = float("nan")
        vp[mask] = float("nan")
    cu_q = torch.tensor(np.concatenate([[0], np.cumsum(lq)]).astype(np.int32), device="cuda")
    return q, kp, vp, cu_q, torch.tensor(lk, dtype=torch.int32, device="cuda"), torch.as_tensor(bt, device="cuda")


def run_paged(q, kp, vp, cu_q, sk, bt, max_lq, W, S, full):
    Tq, Hq, D = q.shape
    out_all = torch.full((Tq * Hq * D + 2 * GUARD,), float("nan"), dtype=torch.bfloat16, device="cuda")
    out = out_all[GUARD:GUARD + Tq * Hq * D].view(Tq, Hq, D)
    lse = torch.full((Hq, Tq), float("nan"), dtype=torch.float32, device="cuda")
    swaa.swaa_prefill_paged(q, kp, vp, out, cu_q, sk, bt, max_lq, W, S, full, lse=lse)
    status = swaa.last_device_status()
    assert torch.isnan(out_all[:GUARD]).all() and torch.isnan(out_all[-GUARD:]).all(), "store outside `out`"
    return out, lse, status


SHAPES = [
    # len_q, len_k, Hq, Hkv, D, page_size
    ((1, 5, 130), (1, 300, 130), 4, 2, 128, 128),
    ((128, 129, 1), (128, 1000, 513), 2, 1, 64, 256),
    ((300,), (1500,), 3, 1, 128, 128),
    ((77, 200), (77 + 128 * 3, 200 + 1), 2, 2, 64, 128),
    ((256, 640), (256 + 64, 640), 8, 2, 128, 384),   # a prompt fed whole (len_q == len_k) next to a chunk
]
POLICIES = [(1, 0, True), (1, 0, False), (128, 0, False), (128, 4, False), (100, 7, False), (129, 130, False),
            (300, 1, False), (4096, 4, False)]


@pytest.mark.parametrize("shape", SHAPES)
def test_paged_prefill_small_shapes(shape):
    lq, lk, Hq, Hkv, D, page = shape
    q, kp, vp, cu_q, sk, bt = make_paged(lq, lk, Hq, Hkv, D, page, seed=700 + sum(lk))
    qh, kh, vh = (inputs.to_f32_numpy(t) for t in (q, kp, vp))
    for W, S, full in POLICIES:
        out, lse, status = run_paged(q, kp, vp, cu_q, sk, bt, max(lq), W, S, full)
        assert status == 0
        ref = oracle.prefill_paged(qh, kh, vh, cu_q.cpu().numpy(), lk, bt.cpu().numpy(), W, S, full)
        check_against_oracle(out, ref["out"], f"paged prefill {shape} W={W} S={S} full={full}")
        np.testing.assert_allclose(lse.cpu().numpy().T, ref["lse"], rtol=0, atol=2e-3)


def test_paged_prefill_long_context_sampled_rows():
    """A 4096-token chunk at the end of a 40000-token paged context, long-context heads and mask."""
    lq, lk, Hq, Hkv, D, W, S, page = (4096,), (40000,), 32, 8, 128, 2048, 4, 256
    q, kp, vp, cu_q, sk, bt = make_paged(lq, lk, Hq, Hkv, D, page, seed=78)
    out, lse, status = run_paged(q, kp, vp, cu_q, sk, bt, lq[0], W, S, False)
    assert status == 0
    rng = np.random.default_rng(3)
    rt = np.concatenate([np.arange(0, 130), np.arange(4096 - 130, 4096), rng.integers(0, 4096, 400)])
    rh = rng.integers(0, Hq, rt.shape[0]).astype(np.int32)
    ref = oracle.prefill_paged(inputs.to_f32_numpy(q), inputs.to_f32_numpy(kp), inputs.to_f32_numpy(vp), [0, lq[0]], lk,
                               bt.cpu().numpy(), W, S, False, rows=(rt, rh))
    got = out[torch.as_tensor(rt, device="cuda"), torch.as_tensor(rh.astype(np.int64), device="cuda")]
    check_against_oracle(got, ref["out"], "paged chunk of a long context")
    assert not torch.isnan(out.float()).any()


@pytest.mark.parametrize("D", [64, 128])
def test_paged_prefill_many_short_sequences_walk_single_tile_ragged_items(D):
    """Many sequences of fewer than 128 keys with several head pairs per kv head: every block walks a run of items
    whose only key tile is ragged, so consecutive tiles in different ring stages each need their rows past the
    sequence end cleared before the product may read them (one cleared-barrier per stage)."""
    rng = np.random.default_rng(17)
    B, Hq, Hkv, page = 96, 8, 2, 128
    lk = tuple(int(x) for x in rng.integers(1, 128, B))
    lq = tuple(int(rng.integers(1, n + 1)) for n in lk)
    q, kp, vp, cu_q, sk, bt = make_paged(lq, lk, Hq, Hkv, D, page, seed=811 + D)
    qh, kh, vh = (inputs.to_f32_numpy(t) for t in (q, kp, vp))
    for W, S, full in ((1, 0, True), (40, 3, False)):
        for _ in range(3):  # the hazard was a matter of timing: run it a few times
            out, lse, status = run_paged(q, kp, vp, cu_q, sk, bt, max(lq), W, S, full)
            assert status == 0
        ref = oracle.prefill_paged(qh, kh, vh, cu_q.cpu().numpy(), lk, bt.cpu().numpy(), W, S, full)
        check_against_oracle(out, ref["out"], f"many short paged sequences D={D} full={full}")


def test_paged_prefill_reports_a_bad_page_index():
    q, kp, vp, cu_q, sk, bt = make_paged((10, 20), (200, 20), 2, 1, 64, 128, seed=9, poison=False)
    bt2 = bt.clone()
    bt2[0, 1] = kp.shape[0] + 3
    out, _, status = run_paged(q, kp, vp, cu_q, sk, bt2, 20, 1, 0, True)
    assert status == -5 and swaa.last_device_status() == 0

"""GPU parity of swaa_prefill_chunked (through the C ABI) against the float64 oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_2512_10411_b200 as swaa
from paper_2512_10411_b200 import inputs
from helpers import check_against_oracle

pytestmark = pytest.mark.gpu

GUARD = 4096  # bf16 elements of NaN canary on each side of `out`


def _randn_bf16(shape, seed):
    g = torch.Generator(device="cuda").manual_seed(seed)
    return torch.randn(shape, generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)


def _cu(lens):
    return torch.tensor(np.concatenate([[0], np.cumsum(lens)]).astype(np.int32), device="cuda")


def run_chunked(q, k, v, lq, lk, W, S, full, scale=0.0):
    Tq, Hq, D = q.shape
    out_all = torch.full((Tq * Hq * D + 2 * GUARD,), float("nan"), dtype=torch.bfloat16, device="cuda")
    out = out_all[GUARD:GUARD + Tq * Hq * D].view(Tq, Hq, D)
    lse = torch.full((Hq, Tq), float("nan"), dtype=torch.float32, device="cuda")
    swaa.swaa_prefill_chunked(q, k, v, out, _cu(lq), _cu(lk), max(lq), max(lk), W, S, full, scale=scale, lse=lse)
    status = swaa.last_device_status()
    assert torch.isnan(out_all[:GUARD]).all() and torch.isnan(out_all[-GUARD:]).all(), "store outside `out`"
    return out, lse, status


def make(lq, lk, Hq, Hkv, D, seed):
    return (_randn_bf16((sum(lq), Hq, D), seed), _randn_bf16((sum(lk), Hkv, D), seed + 1),
            _randn_bf16((sum(lk), Hkv, D), seed + 2))


SHAPES = [
    # len_q per sequence, len_k per sequence, Hq, Hkv, D
    ((1, 5, 130), (1, 300, 130), 4, 2, 128),
    ((128, 129, 1), (128, 1000, 513), 2, 1, 64),
    ((300,), (1500,), 3, 1, 128),          # odd group size
    ((77, 200), (77 + 128 * 3, 200 + 1), 2, 2, 64),
    ((256,), (256 + 64,), 8, 2, 128),      # offset that is not a multiple of the tile size
]
POLICIES = [(1, 0, True), (1, 0, False), (128, 0, False), (128, 4, False), (100, 7, False), (129, 130, False),
            (300, 1, False), (4096, 4, False), (17, 260, False)]


@pytest.mark.parametrize("shape", SHAPES)
def test_chunked_prefill_small_shapes(shape):
    lq, lk, Hq, Hkv, D = shape
    q, k, v = make(lq, lk, Hq, Hkv, D, seed=500 + sum(lk))
    qh, kh, vh = (inputs.to_f32_numpy(t) for t in (q, k, v))
    for W, S, full in POLICIES:
        out, lse, status = run_chunked(q, k, v, lq, lk, W, S, full)
        assert status == 0
        ref = oracle.prefill_chunked(qh, kh, vh, _cu(lq).cpu().numpy(), _cu(lk).cpu().numpy(), W, S, full)
        check_against_oracle(out, ref["out"], f"chunked {shape} W={W} S={S} full={full}")
        np.testing.assert_allclose(lse.cpu().numpy().T, ref["lse"], rtol=0, atol=2e-3)


def test_chunked_prefill_visible_set_is_bit_exact():
    """Q = 0 and one-hot V: out[c] > 0 exactly where key t*D+c is visible to the row, exactly 0 elsewhere."""
    lq, lk, Hq, Hkv, D = (200,), (584,), 2, 1, 64
    q = torch.zeros((lq[0], Hq, D), dtype=torch.bfloat16, device="cuda")
    k = _randn_bf16((lk[0], Hkv, D), 9)
    Lp = ((lk[0] + D - 1) // D) * D
    for W, S, full in ((100, 3, False), (1, 0, False), (64, 70, False), (130, 0, False), (5, 0, True)):
        seen = np.zeros((lq[0], Lp), dtype=bool)
        for t in range(Lp // D):
            v = torch.zeros((lk[0], Hkv, D), dtype=torch.bfloat16, device="cuda")
            idx = torch.arange(t * D, min((t + 1) * D, lk[0]), device="cuda")
            v[idx, :, idx - t * D] = 1.0
            out, _, status = run_chunked(q, k, v, lq, lk, W, S, full)
            assert status == 0
            o = out.float().cpu().numpy()
            assert (o >= 0).all() and np.array_equal(o[:, 0] > 0, o[:, 1] > 0)
            seen[:, t * D:(t + 1) * D] = o[:, 0] > 0
        off = lk[0] - lq[0]
        want = np.array([[j < lk[0] and oracle.visible(off + i, j, W, S, full) for j in range(Lp)] for i in range(lq[0])])
        assert np.array_equal(seen, want), (W, S, full)


def test_chunked_prefill_long_context_sampled_rows():
    """A 4096-token chunk at the end of a 40000-token context, the long-context heads and mask (W=2048, n_sink=4)."""
    lq, lk, Hq, Hkv, D, W, S = (4096,), (40000,), 32, 8, 128, 2048, 4
    q, k, v = make(lq, lk, Hq, Hkv, D, seed=77)
    out, lse, status = run_chunked(q, k, v, lq, lk, W, S, False)
    assert status == 0
    rng = np.random.default_rng(3)
    rt = np.concatenate([np.arange(0, 130), np.arange(4096 - 130, 4096), rng.integers(0, 4096, 600)])
    rh = rng.integers(0, Hq, rt.shape[0]).astype(np.int32)
    ref = oracle.prefill_chunked(inputs.to_f32_numpy(q), inputs.to_f32_numpy(k), inputs.to_f32_numpy(v), [0, lq[0]],
                                 [0, lk[0]], W, S, False, rows=(rt, rh))
    assert (ref["nvis"] == W + S).all()
    got = out[torch.as_tensor(rt, device="cuda"), torch.as_tensor(rh.astype(np.int64), device="cuda")]
    check_against_oracle(got, ref["out"], "chunk of a long context")
    np.testing.assert_allclose(lse.cpu().numpy()[rh, rt], ref["lse"], rtol=0, atol=2e-3)
    assert not torch.isnan(out.float()).any()


def test_chunked_prefill_equal_lengths_match_prefill_bitwise():
    lens = (300, 129)
    q, k, v = make(lens, lens, 4, 2, 128, seed=91)
    a, _, sa = run_chunked(q, k, v, lens, lens, 100, 7, False)
    b = torch.empty_like(q)
    swaa.swaa_prefill(q, k, v, b, _cu(lens), max(lens), 100, 7, False)
    assert sa == 0 and swaa.last_device_status() == 0
    assert torch.equal(a, b)


def test_chunked_prefill_reports_more_queries_than_keys():
    lq, lk = (64, 10), (80, 9)  # the second sequence has more queries than keys
    q, k, v = make(lq, lk, 2, 1, 64, seed=5)
    out, _, status = run_chunked(q, k, v, lq, lk, 16, 0, False)
    assert status == -5
    assert swaa.last_device_status() == 0  # reading clears it
    ref = oracle.prefill_chunked(inputs.to_f32_numpy(q[:64]), inputs.to_f32_numpy(k[:80]), inputs.to_f32_numpy(v[:80]),
                                 [0, 64], [0, 80], 16, 0, False)
    check_against_oracle(out[:64], ref["out"], "valid sequence next to a bad one")
    assert torch.isnan(out[64:].float()).all()  # rows of the bad sequence are not written


def test_lazy_ratio_matches_oracle():
    """Last 64 tokens of two contexts, recent window 1024 (the paper's probe), plus a small ragged case."""
    for lq, lk, Hq, Hkv, D, recent, S in (((64, 64), (3000, 1500), 8, 2, 128, 1024, 0), ((5, 64), (70, 900), 4, 2, 64, 100, 4)):
        q, k, v = make(lq, lk, Hq, Hkv, D, seed=123)
        q = (q.float() * 2.0).to(torch.bfloat16)  # sharper softmax: the ratio is not just a key count
        ratio = torch.full((Hq,), float("nan"), device="cuda")
        sl = torch.empty((2, Hq, sum(lq)), dtype=torch.float32, device="cuda")
        # the probe needs neither values nor an attention output: both may be left out
        swaa.swaa_lazy_ratio(q, k, None, _cu(lq), _cu(lk), max(lq), max(lk), recent, S, ratio, None, sl)
        assert swaa.last_device_status() == 0
        # its two log-sum-exp passes against the oracle's (windowed + sinks, then full causal)
        for idx, (W_, S_, full_) in enumerate(((recent, S, False), (1, 0, True))):
            want = oracle.prefill_chunked(inputs.to_f32_numpy(q), inputs.to_f32_numpy(k), inputs.to_f32_numpy(k),
                                          _cu(lq).cpu().numpy(), _cu(lk).cpu().numpy(), W_, S_, full_)["lse"]
            np.testing.assert_allclose(sl[idx].cpu().numpy().T, want, rtol=0, atol=2e-3)
        ref = oracle.lazy_ratio(inputs.to_f32_numpy(q), inputs.to_f32_numpy(k), None, _cu(lq).cpu().numpy(),
                                _cu(lk).cpu().numpy(), recent, S)
        got = ratio.cpu().numpy()
        assert np.abs(got - ref).max() <= 5e-3, (got, ref)
        assert ((ref > 0.05) & (ref < 0.999)).any()


def test_mixed_batch_with_a_mask_policy_per_sequence():
    """One launch serving prefill chunks under the SWA mask next to single decode tokens under full attention
    (Fig. 1a), dense and paged keys, against the oracle's per-sequence policy."""
    lq, lk = (130, 1, 300, 1, 64), (130, 1700, 900, 129, 64)
    flags = [0, 1, 0, 1, 1]
    fs = torch.tensor(flags, dtype=torch.uint8, device="cuda")
    for Hq, Hkv, D in ((4, 2, 128), (6, 2, 64)):
        q, k, v = make(lq, lk, Hq, Hkv, D, seed=900 + D)
        qh, kh, vh = (inputs.to_f32_numpy(t) for t in (q, k, v))
        for W, S in ((128, 4), (100, 7), (1, 0)):
            Tq = sum(lq)
            out = torch.full((Tq, Hq, D), float("nan"), dtype=torch.bfloat16, device="cuda")
            lse = torch.full((Hq, Tq), float("nan"), dtype=torch.float32, device="cuda")
            swaa.swaa_prefill_chunked(q, k, v, out, _cu(lq), _cu(lk), max(lq), max(lk), W, S, False, lse=lse,
                                      is_full_seq=fs)
            assert swaa.last_device_status() == 0
            ref = oracle.prefill_chunked(qh, kh, vh, _cu(lq).cpu().numpy(), _cu(lk).cpu().numpy(), W, S, False,
                                         is_full_seq=flags)
            check_against_oracle(out, ref["out"], f"mixed batch D={D} W={W} S={S}")
            np.testing.assert_allclose(lse.cpu().numpy().T, ref["lse"], rtol=0, atol=2e-3)
            # the same keys scattered over pages
            page = 128
            blocks = [(n + page - 1) // page for n in lk]
            num_pages = sum(blocks) + 2
            perm = np.random.default_rng(5).permutation(num_pages)
            kp = torch.full((num_pages, page, Hkv, D), float("nan"), dtype=torch.bfloat16, device="cuda")
            vp = torch.full_like(kp, float("nan"))
            bt = np.full((len(lk), max(blocks)), -1, dtype=np.int32)
            cuk = np.concatenate([[0], np.cumsum(lk)])
            nxt = 0
            for b, n in enumerate(lk):
                for blk in range(blocks[b]):
                    pg = int(perm[nxt]); nxt += 1
                    bt[b, blk] = pg
                    m = min(page, n - blk * page)
                    kp[pg, :m] = k[cuk[b] + blk * page:cuk[b] + blk * page + m]
                    vp[pg, :m] = v[cuk[b] + blk * page:cuk[b] + blk * page + m]
            out2 = torch.full_like(out, float("nan"))
            swaa.swaa_prefill_paged(q, kp, vp, out2, _cu(lq), torch.tensor(lk, dtype=torch.int32, device="cuda"),
                                    torch.as_tensor(bt, device="cuda"), max(lq), W, S, False, is_full_seq=fs)
            assert swaa.last_device_status() == 0
            check_against_oracle(out2, ref["out"], f"mixed paged batch D={D} W={W} S={S}")

"""GPU parity of swaa_decode_partial + swaa_decode_combine (through the C ABI) against the float64 oracle.

The participants that would each hold one shard of a cache cut along the context are run one after another on one
GPU; the kernels read their own shard only, so nothing else distinguishes the ranks.  The exchange of the partials
(a gather of B * Hq * (D + 2) floats per participant) is a plain copy here; its collective form is covered on CPU
by tests/test_bench_multirank_cpu.py."""
import numpy as np
import pytest
import torch

import oracle
import paper_2512_10411_b200 as swaa
from paper_2512_10411_b200 import inputs
from helpers import check_against_oracle

pytestmark = pytest.mark.gpu


def run_split(q, kc, vc, sl, cuts, W, S, full, poison=True):
    """Partials of the shards [cuts[r], cuts[r+1]) of every sequence, then the combine.  Each shard is copied into
    a buffer of its own; entries past a sequence's length are poisoned with NaN there."""
    B, Hq, D = q.shape
    Hkv = kc.shape[2]
    parts = torch.full((len(cuts) - 1, B, Hq, D + 2), float("nan"), dtype=torch.float32, device="cuda")
    for r, (a, b) in enumerate(zip(cuts[:-1], cuts[1:])):
        ks, vs = kc[:, a:b].contiguous(), vc[:, a:b].contiguous()
        if poison:
            pos = torch.arange(a, b, device="cuda")[None, :] >= sl[:, None]
            ks[pos] = float("nan")
            vs[pos] = float("nan")
        ws = torch.full((swaa.decode_partial_workspace_size(B, Hq, Hkv, D, b - a, W, S, full),), 0xA5, dtype=torch.uint8,
                        device="cuda")
        swaa.swaa_decode_partial(q, ks, vs, parts[r], sl, a, W, S, full, ws)
        assert swaa.last_device_status() == 0
    out = torch.full((B, Hq, D), float("nan"), dtype=torch.bfloat16, device="cuda")
    swaa.swaa_decode_combine(parts, out)
    assert swaa.last_device_status() == 0
    return parts, out


def check_partials(parts, q, kc, vc, sl, cuts, W, S, full):
    qh, kh, vh = (inputs.to_f32_numpy(t) for t in (q, kc, vc))
    slh = sl.cpu().numpy()
    for r, (a, b) in enumerate(zip(cuts[:-1], cuts[1:])):
        kh_r, vh_r = np.nan_to_num(kh[:, a:b]), np.nan_to_num(vh[:, a:b])
        ref = oracle.decode_partial(qh, kh_r, vh_r, slh, a, W, S, full)["part"]
        got = parts[r].double().cpu().numpy()
        empty = ref[..., 1] == 0
        assert np.array_equal(got[..., 1] == 0, empty), "which rows are empty"
        assert np.isneginf(got[..., 0][empty]).all() and (got[..., 2:][empty] == 0).all()
        ne = ~empty
        if ne.any():
            np.testing.assert_allclose(got[..., 0][ne], ref[..., 0][ne], rtol=0, atol=2e-3)
            # (l, o) relative to their own maximum: compare the log-sum-exp and the normalised output
            np.testing.assert_allclose(got[..., 0][ne] + np.log(got[..., 1][ne]), ref[..., 0][ne] + np.log(ref[..., 1][ne]),
                                       rtol=0, atol=2e-3)
            check_against_oracle(torch.from_numpy(got[..., 2:][ne] / got[..., 1:2][ne]).to(torch.bfloat16),
                                 ref[..., 2:][ne] / ref[..., 1:2][ne], f"partial of shard {r}")


SHAPES = [
    # B, Lmax, Hq, Hkv, D, seqlens
    (3, 3000, 8, 2, 128, (3000, 777, 1)),
    (2, 5000, 4, 4, 64, (4100, 5000)),
    (4, 1500, 32, 2, 128, (1500, 64, 65, 1000)),   # 16 query heads per kv head
    (70, 300, 2, 1, 64, None),                     # many short sequences
]


@pytest.mark.parametrize("shape", SHAPES)
def test_split_decode_small_shapes(shape):
    B, Lmax, Hq, Hkv, D, sl_ = shape
    if sl_ is None:
        sl_ = tuple(int(x) for x in np.random.default_rng(3).integers(1, Lmax + 1, B))
    cfg = inputs.DecodeConfig("split", B, Lmax, Hq, Hkv, D, 0, 0, seed=1400 + B, seqlens=sl_)
    q, kc, vc, sl = inputs.make_decode_inputs(cfg, "cuda")
    qh, kh, vh = (inputs.to_f32_numpy(t) for t in (q, kc, vc))
    for cuts in ((0, Lmax), (0, Lmax // 2, Lmax), (0, 64, 65, 700 if Lmax > 700 else 100, Lmax), (0, 1, Lmax - 1, Lmax)):
        for W, S, full in ((512, 4, False), (1, 0, True), (100, 70, False), (1, 0, False), (4096, 0, False)):
            parts, out = run_split(q, kc, vc, sl, cuts, W, S, full)
            ref = oracle.decode(qh, kh, vh, sl_, W, S, full)
            check_against_oracle(out, ref["out"], f"split decode {shape[:5]} cuts={cuts} W={W} S={S} full={full}")
            check_partials(parts, q, kc, vc, sl, cuts, W, S, full)


@pytest.mark.parametrize("full", [True, False])
@pytest.mark.parametrize("P", [2, 4, 8])
def test_split_decode_full_size_workload(P, full):
    """Workload 4 (B=16, 65536-entry cache, Hq=32, Hkv=8, D=128; SWA: W=4096, n_sink=4) cut into P shards, with ragged
    lengths so that some shards hold nothing of some sequences."""
    sl_ = (65536, 65536, 40000, 8192, 4100, 1, 65535, 30000, 65536, 12345, 16384, 16385, 50000, 2, 65536, 60000)
    cfg = inputs.DecodeConfig("cfg4_split", 16, 65536, 32, 8, 128, 4096, 4, seed=4, seqlens=sl_)
    q, kc, vc, sl = inputs.make_decode_inputs(cfg, "cuda")
    cuts = tuple(65536 * r // P for r in range(P + 1))
    parts, out = run_split(q, kc, vc, sl, cuts, cfg.window, cfg.n_sink, full, poison=False)
    ref = oracle.decode(inputs.to_f32_numpy(q), inputs.to_f32_numpy(kc), inputs.to_f32_numpy(vc), sl_, cfg.window,
                        cfg.n_sink, full)
    r = check_against_oracle(out, ref["out"], f"cfg4 split P={P} full={full}")
    print(f"cfg4 split over {P} shards, full={full}: max abs err {r[0]:.3e}, max rel err {r[1]:.3e}")


def test_split_decode_argument_errors_and_bad_lengths():
    cfg = inputs.DecodeConfig("splitbad", 2, 256, 4, 2, 64, 0, 0, seed=5, seqlens=(256, 100))
    q, kc, vc, sl = inputs.make_decode_inputs(cfg, "cuda")
    part = torch.empty((2, 4, 66), dtype=torch.float32, device="cuda")
    ws = torch.empty(swaa.decode_partial_workspace_size(2, 4, 2, 64, 256, 16, 0, False), dtype=torch.uint8, device="cuda")
    with pytest.raises(swaa.SwaaError) as e:
        swaa.swaa_decode_partial(q, kc, vc, part, sl, 0, 0, 0, False, ws)      # window < 1
    assert e.value.status == -1
    with pytest.raises(swaa.SwaaError) as e:
        swaa.swaa_decode_partial(q, kc, vc, part, sl, -1, 16, 0, False, ws)    # negative position
    assert e.value.status == -1
    with pytest.raises(swaa.SwaaError) as e:
        swaa.swaa_decode_partial(q, kc, vc, part, sl, 0, 16, 0, False, ws[:64])
    assert e.value.status == -4
    bad = torch.tensor([256, 0], dtype=torch.int32, device="cuda")
    swaa.swaa_decode_partial(q, kc, vc, part, bad, 0, 16, 0, False, ws)
    assert swaa.last_device_status() == -5
    swaa.swaa_decode_partial(q, kc, vc, part, sl, 0, 16, 0, False, ws)
    assert swaa.last_device_status() == 0

"""GPU parity of swaa_prefill_context_parallel (through the C ABI) against the float64 oracle.

The participants of a context-parallel prefill are emulated one after another on one GPU: each gets its stretch of
every sequence, the halo of window - 1 earlier keys and the sink rows, exactly what a neighbour copy and a broadcast
would have put into its memory; the kernels read local memory only, so nothing else distinguishes the ranks."""
import numpy as np
import pytest
import torch

import oracle
import paper_2512_10411_b200 as swaa
from paper_2512_10411_b200 import inputs
from helpers import check_against_oracle

pytestmark = pytest.mark.gpu


def split(q, k, v, lens, r, P, W, S, halo=None):
    """Inputs of participant r of P: (q_r, k_local, v_local, sink_k, sink_v, lq, lk, key_pos0, owned packed rows)."""
    cu = np.concatenate([[0], np.cumsum(lens)])
    qs, ks, vs, lq, lk, p0, rows = [], [], [], [], [], [], []
    for b, n in enumerate(lens):
        own0, own1 = n * r // P, n * (r + 1) // P
        h0 = max(0, own0 - (W - 1 if halo is None else halo))
        qs.append(q[cu[b] + own0:cu[b] + own1]); ks.append(k[cu[b] + h0:cu[b] + own1]); vs.append(v[cu[b] + h0:cu[b] + own1])
        lq.append(own1 - own0); lk.append(own1 - h0); p0.append(h0)
        rows.append(np.arange(cu[b] + own0, cu[b] + own1))
    sink_rows = max(S, 1)
    B, Hkv, D = len(lens), k.shape[1], k.shape[2]
    sk = torch.zeros((B, sink_rows, Hkv, D), dtype=torch.bfloat16, device="cuda")
    sv = torch.zeros_like(sk)
    for b, n in enumerate(lens):
        m = min(sink_rows, n)
        sk[b, :m] = k[cu[b]:cu[b] + m]
        sv[b, :m] = v[cu[b]:cu[b] + m]
    return torch.cat(qs), torch.cat(ks), torch.cat(vs), sk, sv, lq, lk, p0, np.concatenate(rows)


def _cu(lens):
    return torch.tensor(np.concatenate([[0], np.cumsum(lens)]).astype(np.int32), device="cuda")


def run_cp(qr, kl, vl, sk, sv, lq, lk, p0, W, S):
    Tq, Hq, D = qr.shape
    out = torch.full((Tq, Hq, D), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((Hq, Tq), float("nan"), dtype=torch.float32, device="cuda")
    swaa.swaa_prefill_context_parallel(qr, kl, vl, sk, sv, out, _cu(lq), _cu(lk),
                                       torch.tensor(p0, dtype=torch.int32, device="cuda"), max(lq), max(lk), W, S,
                                       lse=lse)
    return out, lse, swaa.last_device_status()


@pytest.mark.parametrize("shape", [((700, 300, 129), 4, 2, 128), ((1000,), 2, 1, 64), ((515, 256), 6, 2, 128)])
@pytest.mark.parametrize("P", [2, 3])
def test_context_parallel_small_ragged_shapes(shape, P):
    lens, Hq, Hkv, D = shape
    cfg = inputs.PrefillConfig("cp", lens, Hq, Hkv, D, 1, 0, False, seed=1200 + P)
    q, k, v, _ = inputs.make_prefill_inputs(cfg, "cuda")
    for W, S in ((128, 4), (100, 7), (1, 0), (129, 130), (64, 300), (4096, 2)):
        for r in range(P):
            qr, kl, vl, sk, sv, lq, lk, p0, rows = split(q, k, v, lens, r, P, W, S)
            if sum(lq) == 0:
                continue
            out, lse, status = run_cp(qr, kl, vl, sk, sv, lq, lk, p0, W, S)
            assert status == 0
            ref = oracle.prefill_cp(inputs.to_f32_numpy(qr), inputs.to_f32_numpy(kl), inputs.to_f32_numpy(vl),
                                    inputs.to_f32_numpy(sk), inputs.to_f32_numpy(sv), _cu(lq).cpu().numpy(),
                                    _cu(lk).cpu().numpy(), p0, W, S, False)
            check_against_oracle(out, ref["out"], f"cp {shape} P={P} r={r} W={W} S={S}")
            np.testing.assert_allclose(lse.cpu().numpy().T, ref["lse"], rtol=0, atol=2e-3)


@pytest.mark.parametrize("P", [2, 4])
def test_context_parallel_long_context_workload(P):
    """Workload 2's shape (L=32768, Hq=32, Hkv=8, D=128, W=2048, n_sink=4) cut over P participants run in sequence:
    sampled rows against the oracle's one-shot prefill of the whole sequence, and, with Q = 0, the number of keys every
    row of every participant saw against the closed form (bit-exact visible-set size)."""
    cfg = inputs.cfg_long()
    L, W, S = cfg.seqlens[0], cfg.window, cfg.n_sink
    q, k, v, _ = inputs.make_prefill_inputs(cfg, "cuda")
    qh, kh, vh = (inputs.to_f32_numpy(t) for t in (q, k, v))
    rng = np.random.default_rng(77 + P)
    i = np.arange(L, dtype=np.int64)
    counts = np.minimum(i + 1, W) + np.clip(i - W + 1, 0, S)
    for r in range(P):
        qr, kl, vl, sk, sv, lq, lk, p0, rows = split(q, k, v, (L,), r, P, W, S)
        out, lse, status = run_cp(qr, kl, vl, sk, sv, lq, lk, p0, W, S)
        assert status == 0 and not torch.isnan(out.float()).any()
        n = lq[0]
        loc = np.unique(np.concatenate([np.arange(0, 130), np.arange(n - 130, n), rng.integers(0, n, 300)]))
        rh = rng.integers(0, cfg.Hq, loc.shape[0]).astype(np.int32)
        ref = oracle.prefill(qh, kh, vh, [0, L], W, S, False, rows=(rows[loc], rh))
        got = out[torch.from_numpy(loc).cuda(), torch.from_numpy(rh.astype(np.int64)).cuda()]
        check_against_oracle(got, ref["out"], f"cp cfg2 P={P} r={r}")
        np.testing.assert_allclose(lse.cpu().numpy()[rh, loc], ref["lse"], rtol=0, atol=2e-3)
        out0, lse0, status = run_cp(torch.zeros_like(qr), kl, vl, sk, sv, lq, lk, p0, W, S)
        assert status == 0
        want = torch.from_numpy(counts[rows]).cuda().double()
        assert torch.equal(torch.round(torch.exp(lse0.double())), want[None, :].expand(cfg.Hq, -1)), (P, r)


def test_context_parallel_rejects_a_short_halo_and_argument_errors():
    lens, Hq, Hkv, D, W, S = (600,), 4, 2, 128, 128, 4
    cfg = inputs.PrefillConfig("cpbad", lens, Hq, Hkv, D, W, S, False, seed=1300)
    q, k, v, _ = inputs.make_prefill_inputs(cfg, "cuda")
    qr, kl, vl, sk, sv, lq, lk, p0, rows = split(q, k, v, lens, 1, 2, W, S, halo=50)   # 50 < W - 1 keys of halo
    out, lse, status = run_cp(qr, kl, vl, sk, sv, lq, lk, p0, W, S)
    assert status == -5 and torch.isnan(out.float()).all()
    qr, kl, vl, sk, sv, lq, lk, p0, rows = split(q, k, v, lens, 1, 2, W, S)
    out, lse, status = run_cp(qr, kl, vl, sk[:, :2].contiguous(), sv[:, :2].contiguous(), lq, lk, p0, W, S)  # 2 sink rows < n_sink
    assert status == -5
    out, lse, status = run_cp(qr, kl, vl, sk, sv, lq, lk, p0, W, S)
    assert status == 0
    with pytest.raises(swaa.SwaaError) as e:   # window < 1
        swaa.swaa_prefill_context_parallel(qr, kl, vl, sk, sv, out, _cu(lq), _cu(lk),
                                           torch.tensor(p0, dtype=torch.int32, device="cuda"), max(lq), max(lk), 0, S)
    assert e.value.status == -1

"""GPU parity of swaa_prefill_backward (through the C ABI) against the float64 oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_2512_10411_b200 as swaa
from paper_2512_10411_b200 import inputs
from helpers import ABS_TOL

# Relative bound for gradients.  The forward bound (2e-2) does not carry over: delta_i = dO_i . out_i is taken
# from the bf16 output, and for a row with few visible keys (|out_i| as large as |v|) its error, about
# 2^-9 * sum_d |dO_id out_id|, reaches a few per cent of dP_ij - delta_i, hence of that row's dq.
GRAD_REL_TOL = 5e-2

pytestmark = pytest.mark.gpu


def check_grad(got_bf16, ref, what, slack=None):
    """|err| <= 2e-2 * max(1, largest |ref| of the row), and |err| <= 5e-2 relative to max(|ref|, largest |ref| of the element's row, RMS of
    the tensor).

    Every element of a gradient row is a sum over the same bf16-rounded factors (P_ij for dv, dS_ij = P (dP - delta)
    for dq and dk, the latter up to ~10 for rows with few visible keys) times different channels, and the terms
    cancel (sum_j dS_ij = 0), so the rounding error of an element scales with the row's largest entries rather than
    with the element or the row's RMS.  The row term delta_i = dO_i . out_i is taken from the bf16 output, which puts
    an error of about 2^-9 |dO_i| |out_i| * scale * |k| (a few 1e-3, independent of how small the row's own gradient
    is) on dq and dk; rows whose gradient is tiny or vanishes by cancellation are therefore measured against the
    RMS of the whole tensor.  `slack` (dq only) is an absolute allowance per row for exactly that term, see
    delta_slack()."""
    got = got_bf16.detach().cpu().to(torch.float64).numpy()
    assert np.isfinite(got).all(), f"{what}: non-finite"
    err = np.abs(got - ref)
    rowmax = np.abs(ref).max(axis=-1, keepdims=True)
    floor = np.maximum(np.maximum(np.abs(ref), rowmax), max(np.sqrt((ref ** 2).mean()), 1e-3))  # 1e-3: a gradient that is identically zero (window 1)
    if slack is not None:
        err = np.maximum(err - slack, 0.0)
    rel = err / floor
    # gradients of sink keys add up hundreds of rows and exceed 1, where bf16 rounding alone passes 2e-2 absolute
    absr = err / np.maximum(1.0, rowmax)
    assert absr.max() <= ABS_TOL, f"{what}: max abs err {absr.max():.4g} (relative to max(1, largest |ref| of the row))"
    assert rel.max() <= GRAD_REL_TOL, f"{what}: max rel err {rel.max():.4g}"
    return float(err.max()), float(rel.max())


def delta_slack(out_bf16, dout_bf16, k_bf16, scale):
    """Allowance on dq rows for the rounding of `out`: the kernel (like every flash-style backward) takes
    delta_i = dO_i . out_i from the bf16 output, whose channels carry independent relative errors of up to 2^-9, so
    delta_i is off by about 2^-9 * sqrt(sum_d (dO_id out_id)^2) (three standard deviations allowed), and
    dq_i = scale * sum_j p_ij (dP_ij - delta_i) k_j moves by scale * |error of delta_i| * |sum_j p_ij k_j|, the last
    factor bounded by the largest |k|.  It matters for rows that see two or three keys, where dP_ij - delta_i is a
    small difference of numbers near 10."""
    prod = out_bf16.double() * dout_bf16.double()
    e = 3.0 * 2.0 ** -9 * prod.pow(2).sum(-1, keepdim=True).sqrt()
    return (scale * e * float(k_bf16.abs().max())).cpu().numpy()


def run_forward_backward(cfg, scale=0.0):
    q, k, v, cu = inputs.make_prefill_inputs(cfg, "cuda")
    g = torch.Generator(device="cuda").manual_seed(cfg.seed + 999)
    dout = torch.randn(q.shape, generator=g, device="cuda").to(torch.bfloat16)
    T, Hq, D = q.shape
    out = torch.empty_like(q)
    lse = torch.empty((Hq, T), dtype=torch.float32, device="cuda")
    swaa.swaa_prefill(q, k, v, out, cu, max(cfg.seqlens), cfg.window, cfg.n_sink, cfg.is_full, scale=scale, lse=lse)
    nbytes = swaa.prefill_backward_workspace_size(len(cfg.seqlens), T, Hq, cfg.Hkv, D, cfg.n_sink)
    guard = 4096
    ws_all = torch.full((nbytes + 2 * guard,), 0xA5, dtype=torch.uint8, device="cuda")
    ws = ws_all[guard:guard + nbytes]
    dq = torch.full_like(q, float("nan"))
    dk = torch.full_like(k, float("nan"))
    dv = torch.full_like(v, float("nan"))
    swaa.swaa_prefill_backward(q, k, v, out, dout, lse, cu, max(cfg.seqlens), cfg.window, cfg.n_sink, cfg.is_full, dq, dk,
                               dv, ws, scale=scale)
    assert swaa.last_device_status() == 0
    assert (ws_all[:guard] == 0xA5).all() and (ws_all[-guard:] == 0xA5).all(), "store outside the workspace"
    ref = oracle.prefill_backward_c(inputs.to_f32_numpy(q), inputs.to_f32_numpy(k), inputs.to_f32_numpy(v),
                                    inputs.to_f32_numpy(dout), cu.cpu().numpy(), cfg.window, cfg.n_sink, cfg.is_full,
                                    scale=(scale if scale > 0 else None))
    sl = delta_slack(out, dout, k, scale if scale > 0 else 1.0 / np.sqrt(D))
    worst = [check_grad(t, ref[n], f"{cfg.name} {n}", slack=(sl if n == "dq" else None))
             for n, t in (("dq", dq), ("dk", dk), ("dv", dv))]
    return worst


SMALL = [
    # seqlens, Hq, Hkv, D
    ((300, 1, 129, 128, 517), 4, 2, 128),
    ((1000,), 2, 1, 64),
    ((257, 640), 3, 1, 128),   # three query heads per kv head
    ((200, 333), 2, 2, 64),
    ((63,), 8, 2, 128),
    ((40, 64, 65, 200), 2, 2, 128),  # one query head per kv head: blocks with a single step
    ((130, 1), 8, 1, 128),           # eight query heads per kv head
]
POLICIES = [(1, 0, True), (1, 0, False), (64, 0, False), (128, 4, False), (100, 7, False), (65, 70, False),
            (300, 1, False), (4096, 4, False)]


@pytest.mark.parametrize("shape", SMALL)
def test_backward_small_ragged_shapes(shape):
    seqlens, Hq, Hkv, D = shape
    for idx, (W, S, full) in enumerate(POLICIES):
        run_forward_backward(inputs.PrefillConfig(f"bwd{shape}W{W}S{S}f{full}", seqlens, Hq, Hkv, D, W, S, full,
                                                  seed=300 + idx))


def test_backward_explicit_scale():
    # scale 1/8 instead of the default 1/sqrt(128): sharper softmax, larger dS (whose bf16 rounding sets the error)
    run_forward_backward(inputs.PrefillConfig("bwdscale", (384, 100), 4, 2, 128, 64, 2, False, seed=31), scale=0.125)


def test_backward_tiny_workload():
    """Workload 1 (L=1024, Hq=4, Hkv=2, D=64, W=128, n_sink=4), every gradient element."""
    w = run_forward_backward(inputs.cfg_tiny())
    print("cfg1 backward: (max abs, max rel) for dq, dk, dv:", w)


def test_backward_mid_size_long_window():
    """L=6144, Hq=8, Hkv=2, D=128, W=2048, n_sink=4: several key tiles per band, sinks seen by every later tile."""
    run_forward_backward(inputs.PrefillConfig("bwdmid", (6144,), 8, 2, 128, 2048, 4, False, seed=77))


def test_backward_split_sink_tiles_ragged_batch():
    """Sequences of 4500, 2300 and 70 tokens with 100 sink tokens (two sink key tiles) and W=256: the long sequences
    take the path where a sink tile's query range is cut over several blocks and dk, dv are summed in fp32; the
    short one ends inside the first sink tile, and the second chunk of the 2300-token sequence is partly empty."""
    run_forward_backward(inputs.PrefillConfig("bwdsplit", (4500, 2300, 70), 4, 2, 128, 256, 100, False, seed=91))


@pytest.mark.parametrize("D", [64, 128])
def test_backward_reports_bad_cu_seqlens_and_argument_errors(D):
    """Both kernels: a cu_seqlens that runs past T is reported through the status word and the call returns; host-side
    checks (workspace too small, unsupported head size, window < 1) are refused before any launch."""
    cfg = inputs.PrefillConfig("bwdbad", (256, 256), 4, 2, D, 16, 2, False, seed=63)
    q, k, v, cu = inputs.make_prefill_inputs(cfg, "cuda")
    T, Hq, _ = q.shape
    out, dout = torch.zeros_like(q), torch.ones_like(q)
    lse = torch.zeros((Hq, T), dtype=torch.float32, device="cuda")
    dq, dk, dv = torch.zeros_like(q), torch.zeros_like(k), torch.zeros_like(v)
    ws = torch.empty(swaa.prefill_backward_workspace_size(2, T, Hq, cfg.Hkv, D, 2), dtype=torch.uint8, device="cuda")
    assert swaa.last_device_status() == 0
    bad = torch.tensor([0, 300, 600], dtype=torch.int32, device="cuda")  # second sequence ends past T = 512
    swaa.swaa_prefill_backward(q, k, v, out, dout, lse, bad, 300, 16, 2, False, dq, dk, dv, ws)
    assert swaa.last_device_status() == -5
    swaa.swaa_prefill_backward(q, k, v, out, dout, lse, cu, 256, 16, 2, False, dq, dk, dv, ws)
    assert swaa.last_device_status() == 0
    with pytest.raises(swaa.SwaaError) as e:
        swaa.swaa_prefill_backward(q, k, v, out, dout, lse, cu, 256, 16, 2, False, dq, dk, dv, ws[:1024])
    assert e.value.status == -4
    with pytest.raises(swaa.SwaaError) as e:
        swaa.swaa_prefill_backward(q, k, v, out, dout, lse, cu, 256, 0, 2, False, dq, dk, dv, ws)
    assert e.value.status == -1

"""GPU parity of swaa_prefill_backward (through the C ABI) against the float64 oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_2512_10411_b200 as swaa
from paper_2512_10411_b200 import inputs
from helpers import ABS_TOL

# Tolerance of the gradients: |err| <= 2e-2 * max(|ref|, largest |ref| of the element's row, 1e-2).
#
# Every element of a gradient row is a sum over the same bf16-rounded factors (P_ij for dv; dS_ij = P_ij (dP_ij - delta_i)
# for dq and dk) times different channels, each factor carrying a relative rounding error of at most 2^-9, and the
# terms cancel (sum_j dS_ij = 0): the error of an element therefore scales with the row's largest entries, not with
# the element itself, which is why the relative error is floored at the row's largest |ref|.  The constant 1e-2
# covers gradients that vanish identically (window 1: one key per row, dS = 0) where only rounding noise is left.
# Observed worst cases over all tests of this file: dq 6.9e-3, dk 6.5e-3, dv 7.1e-3 against the gradient for the
# given forward output; dk 8.7e-3 and dv 7.1e-3 against the exact gradient.
#
# What is compared.  swaa_prefill_backward receives the forward output `out` as an argument and forms the row term
# delta_i = dout_i . out_i from it (it never sees the probabilities of a whole row at once).  `out` is bf16, so
# delta_i differs from the exact sum_j p_ij dP_ij by up to 2^-9 sum_d |dout_id out_id|, which moves dq_i by exactly
# -scale * (error of delta_i) * sum_j p_ij k_j (the oracle's pin states and checks this closed form).  For rows that
# see two or three keys that is several per cent of dq (7 % observed), for ordinary rows 1e-3.  The reference for
# all three gradients is therefore the oracle's gradient FOR THE SAME `out` (out_given), at the tolerance above; dk
# and dv, on which the row term acts through sums over many rows, are checked against the exact gradient as well.
# `out` and `lse` handed to the kernel are the oracle's forward result (rounded to bf16 / float32), so these tests do
# not depend on the forward kernel; test_backward_after_the_forward_kernel runs the two kernels back to back.
GRAD_TOL = 2e-2
GRAD_FLOOR = 1e-2

pytestmark = pytest.mark.gpu


def check_grad(got_bf16, ref, what):
    got = got_bf16.detach().cpu().to(torch.float64).numpy()
    assert np.isfinite(got).all(), f"{what}: non-finite"
    err = np.abs(got - ref)
    rowmax = np.abs(ref).max(axis=-1, keepdims=True)
    rel = err / np.maximum(np.maximum(np.abs(ref), rowmax), GRAD_FLOOR)
    assert rel.max() <= GRAD_TOL, f"{what}: max rel err {rel.max():.4g} (abs {err.max():.4g})"
    return float(rel.max())


def oracle_forward(q, k, v, cu, cfg, scale):
    """The oracle's forward pass as the kernel's `out` (bf16) and `lse` (float32, [Hq, T]) arguments."""
    fwd = oracle.prefill(inputs.to_f32_numpy(q), inputs.to_f32_numpy(k), inputs.to_f32_numpy(v), cu.cpu().numpy(),
                         cfg.window, cfg.n_sink, cfg.is_full, scale=(scale if scale > 0 else None))
    out = torch.from_numpy(fwd["out"]).to(torch.bfloat16).cuda()
    lse = torch.from_numpy(np.ascontiguousarray(fwd["lse"].T)).to(torch.float32).cuda()
    return out, lse


def run_forward_backward(cfg, scale=0.0, forward_on_gpu=False):
    q, k, v, cu = inputs.make_prefill_inputs(cfg, "cuda")
    g = torch.Generator(device="cuda").manual_seed(cfg.seed + 999)
    dout = torch.randn(q.shape, generator=g, device="cuda").to(torch.bfloat16)
    T, Hq, D = q.shape
    if forward_on_gpu:
        out = torch.empty_like(q)
        lse = torch.empty((Hq, T), dtype=torch.float32, device="cuda")
        swaa.swaa_prefill(q, k, v, out, cu, max(cfg.seqlens), cfg.window, cfg.n_sink, cfg.is_full, scale=scale, lse=lse)
    else:
        out, lse = oracle_forward(q, k, v, cu, cfg, scale)
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
    args = (inputs.to_f32_numpy(q), inputs.to_f32_numpy(k), inputs.to_f32_numpy(v), inputs.to_f32_numpy(dout),
            cu.cpu().numpy(), cfg.window, cfg.n_sink, cfg.is_full)
    exact = oracle.prefill_backward_c(*args, scale=(scale if scale > 0 else None))
    worst = {}
    if not forward_on_gpu:
        given = oracle.prefill_backward_c(*args, scale=(scale if scale > 0 else None), out_given=inputs.to_f32_numpy(out))
        for n, t in (("dq", dq), ("dk", dk), ("dv", dv)):
            worst[n] = check_grad(t, given[n], f"{cfg.name} {n} (gradient for the given out)")
    else:
        # rows that see at least 32 keys: there the bf16 rounding of `out` moves dq by well under the tolerance
        cu_h = cu.cpu().numpy()
        keep = np.concatenate([np.arange(n) >= 31 for n in np.diff(cu_h)])
        if not cfg.is_full and cfg.window + cfg.n_sink < 32:
            keep[:] = False
        idx = torch.from_numpy(np.nonzero(keep)[0]).cuda()
        if len(idx):
            worst["dq"] = check_grad(dq[idx], exact["dq"][keep], f"{cfg.name} dq (exact, rows with >= 32 keys)")
    for n, t in (("dk", dk), ("dv", dv)):
        worst[n + " exact"] = check_grad(t, exact[n], f"{cfg.name} {n} (exact gradient)")
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
    print("cfg1 backward, worst relative error:", w)


@pytest.mark.parametrize("cfg", [inputs.cfg_tiny(),
                                 inputs.PrefillConfig("fwdbwd128", (700, 130), 8, 2, 128, 256, 4, False, seed=93)])
def test_backward_after_the_forward_kernel(cfg):
    """The two kernels back to back, as a training step runs them: `out` and `lse` come from swaa_prefill.  dk and dv
    against the exact gradient, dq against the exact gradient on the rows that see at least 32 keys."""
    w = run_forward_backward(cfg, forward_on_gpu=True)
    print(f"{cfg.name} forward + backward on the GPU, worst relative error:", w)


def test_backward_mid_size_long_window():
    """L=6144, Hq=8, Hkv=2, D=128, W=2048, n_sink=4: several key tiles per band, sinks seen by every later tile."""
    run_forward_backward(inputs.PrefillConfig("bwdmid", (6144,), 8, 2, 128, 2048, 4, False, seed=77))


def test_backward_split_sink_tiles_ragged_batch():
    """Sequences of 4500, 2300 and 70 tokens with 100 sink tokens (two sink key tiles) and W=256: the long sequences
    take the path where a sink tile's query range is cut over several blocks and dk, dv are summed in fp32; the
    short one ends inside the first sink tile, and the second chunk of the 2300-token sequence is partly empty."""
    run_forward_backward(inputs.PrefillConfig("bwdsplit", (4500, 2300, 70), 4, 2, 128, 256, 100, False, seed=91))


def test_backward_long_context_workload_sampled_rows_and_keys():
    """Workload 2 (L=32768, Hq=32, Hkv=8, D=128, W=2048, n_sink=4, K row 0 shifted) -- the size the benchmark times,
    with 16 chunks per sink key tile.  dq on all boundary rows (first tile, around n_sink, W, W + n_sink, the tail) of
    two heads plus 1024 seeded (row, head) pairs; dk, dv on the sink keys, the same boundaries and 1024 seeded keys of
    one kv head (its row statistics are shared by all of them) plus one seeded 128-key block of every other kv head.
    `out` and `lse` of every row that one of those gradients depends on are the oracle's; the other rows are filled by
    the forward kernel (the backward kernel needs all of them as input, the compared gradients do not depend on them)."""
    cfg = inputs.cfg_long()
    L, W, S = cfg.seqlens[0], cfg.window, cfg.n_sink
    q, k, v, cu = inputs.make_prefill_inputs(cfg, "cuda")
    g = torch.Generator(device="cuda").manual_seed(cfg.seed + 999)
    dout = torch.randn(q.shape, generator=g, device="cuda").to(torch.bfloat16)
    T, Hq, D = q.shape
    G = Hq // cfg.Hkv
    rng = np.random.default_rng(2026)
    pos = set(range(0, 130)) | set(range(L - 130, L))
    for c in (S, W, W + S, L // 2):
        pos |= set(range(max(0, c - 3), min(L, c + 4)))
    pos = np.array(sorted(pos), dtype=np.int64)
    qt = np.concatenate([pos, pos, rng.integers(0, L, 1024)])
    qh = np.concatenate([np.full(len(pos), 0), np.full(len(pos), Hq - 1), rng.integers(0, Hq, 1024)]).astype(np.int32)
    hk_a = int(rng.integers(0, cfg.Hkv))
    kt = [pos, rng.integers(0, L, 1024)]
    kh = [np.full(len(pos), hk_a), np.full(1024, hk_a)]
    need = np.zeros((T, Hq), dtype=bool)          # rows whose out / lse some compared gradient depends on
    need[qt, qh] = True
    need[:, hk_a * G:(hk_a + 1) * G] = True       # the sink keys of this head are seen by every row
    for hk in range(cfg.Hkv):
        if hk != hk_a:
            j0 = int(rng.integers(S, L - 128))
            kt.append(np.arange(j0, j0 + 128))
            kh.append(np.full(128, hk))
            need[j0:min(L, j0 + 128 + W), hk * G:(hk + 1) * G] = True
    kt, kh = np.concatenate(kt).astype(np.int64), np.concatenate(kh).astype(np.int32)
    qf, kf, vf, df = (inputs.to_f32_numpy(t) for t in (q, k, v, dout))
    nt, nh = np.nonzero(need)
    fwd = oracle.prefill(qf, kf, vf, [0, L], W, S, False, rows=(nt, nh.astype(np.int32)))
    out = torch.empty_like(q)
    lse = torch.empty((Hq, T), dtype=torch.float32, device="cuda")
    swaa.swaa_prefill(q, k, v, out, cu, L, W, S, False, lse=lse)   # filler for the rows nothing compared depends on
    nti, nhi = torch.from_numpy(nt).cuda(), torch.from_numpy(nh).cuda()
    out[nti, nhi] = torch.from_numpy(fwd["out"]).to(torch.bfloat16).cuda()
    lse[nhi, nti] = torch.from_numpy(fwd["lse"]).to(torch.float32).cuda()
    ws = torch.empty(swaa.prefill_backward_workspace_size(1, T, Hq, cfg.Hkv, D, S), dtype=torch.uint8, device="cuda")
    dq, dk, dv = torch.full_like(q, float("nan")), torch.full_like(k, float("nan")), torch.full_like(v, float("nan"))
    swaa.swaa_prefill_backward(q, k, v, out, dout, lse, cu, L, W, S, False, dq, dk, dv, ws)
    assert swaa.last_device_status() == 0
    for name, t in (("dq", dq), ("dk", dk), ("dv", dv)):
        assert torch.isfinite(t.float()).all(), f"{name}: some element was not written"
    og = np.zeros((T, Hq, D), dtype=np.float32)
    og[nt, nh] = torch.from_numpy(fwd["out"]).to(torch.bfloat16).to(torch.float32).numpy()
    given = oracle.prefill_backward_rows(qf, kf, vf, df, [0, L], W, S, False, (qt, qh), (kt, kh), out_given=og)
    qti, qhi = torch.from_numpy(qt).cuda(), torch.from_numpy(qh.astype(np.int64)).cuda()
    kti, khi = torch.from_numpy(kt).cuda(), torch.from_numpy(kh.astype(np.int64)).cuda()
    w = [check_grad(dq[qti, qhi], given["dq"], "cfg2 dq"), check_grad(dk[kti, khi], given["dk"], "cfg2 dk"),
         check_grad(dv[kti, khi], given["dv"], "cfg2 dv")]
    print(f"cfg2 backward, {len(qt)} rows and {len(kt)} keys: worst relative error of dq, dk, dv:", w)


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
    # sequences longer than the stated max_seqlen: reported like the forward pass does, dk and dv rows untouched
    dk.fill_(float("nan"))
    dv.fill_(float("nan"))
    swaa.swaa_prefill_backward(q, k, v, out, dout, lse, cu, 128, 16, 2, False, dq, dk, dv, ws)
    assert swaa.last_device_status() == -5
    assert torch.isnan(dk.float()).all() and torch.isnan(dv.float()).all() and (dq == 0).all()
    swaa.swaa_prefill_backward(q, k, v, out, dout, lse, cu, 256, 16, 2, False, dq, dk, dv, ws)
    assert swaa.last_device_status() == 0
    with pytest.raises(swaa.SwaaError) as e:
        swaa.swaa_prefill_backward(q, k, v, out, dout, lse, cu, 256, 16, 2, False, dq, dk, dv, ws[:1024])
    assert e.value.status == -4
    with pytest.raises(swaa.SwaaError) as e:
        swaa.swaa_prefill_backward(q, k, v, out, dout, lse, cu, 256, 0, 2, False, dq, dk, dv, ws)
    assert e.value.status == -1

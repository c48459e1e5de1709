"""Pins for the float64 CPU oracle: it is checked against what the paper and the mathematics fix,
never against itself.  All CPU-only.

Each test is chosen so that one plausible mistake in the oracle fails it: an off-by-one window
(W vs W+1 keys), sinks taken relative to the packed buffer instead of each sequence, a dropped or
double-counted sink/window overlap, a wrong GQA head map, a missing scale, K and V swapped, a softmax
that is not normalised, a decode query placed at the wrong position.
"""
import itertools
import os

import numpy as np
import pytest
import torch

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _bf16_randn(shape, seed):
    g = torch.Generator().manual_seed(seed)
    return torch.randn(shape, generator=g).to(torch.bfloat16).to(torch.float32).numpy()


def _range_union_visible(i, W, S, is_full):
    """The mask stated as a union of index ranges (Sec. 3.2.1: local window AND the first k tokens;
    the window holds W keys ending at the query itself), not as the oracle's predicate."""
    if is_full:
        return set(range(0, i + 1))
    window = set(range(max(0, i - W + 1), i + 1))
    sinks = set(range(0, min(S, i + 1)))
    return window | sinks


GRID = [(L, W, S) for L in (1, 2, 7, 33, 64) for W in (1, 2, 5, 8, 64, 100) for S in (0, 1, 2, 9, 70)]


@pytest.mark.parametrize("is_full", [False, True])
def test_visible_set_matches_range_union_bruteforce(is_full):
    for L, W, S in GRID:
        for i in range(L):
            want = _range_union_visible(i, W, S, is_full)
            got = {j for j in range(-1, L + 1) if oracle.visible(i, j, W, S, is_full)}
            assert got == want, (L, W, S, i)


def test_pair_count_closed_form_fixture():
    with open(os.path.join(GOLDEN, "visible_pair_counts.txt")) as f:
        rows = [ln for ln in f if ln.strip() and not ln.startswith("#")]
    assert len(rows) >= 6
    for ln in rows:
        L, W, S, full, want = (int(x) for x in ln.split(";"))
        if L > 4096:
            continue  # enumeration is quadratic; the large entry is checked through nvis below
        assert oracle.count_pairs(L, W, S, bool(full)) == want, ln


def test_pair_count_closed_form_grid():
    for L, W, S in itertools.product((40, 97), (1, 3, 16), (0, 1, 5, 20)):
        if L < W + S:
            continue
        closed = W * (W + 1) // 2 + (L - W) * W + S * (S + 1) // 2 + (L - W - S) * S
        assert oracle.count_pairs(L, W, S, False) == closed
        assert oracle.count_pairs(L, W, S, True) == L * (L + 1) // 2


def _sdpa_f64(q, k, v, mask=None, causal=False, scale=None):
    """Library routine: torch float64 scaled_dot_product_attention on [H, L, D] tensors."""
    qt = torch.from_numpy(q).double().permute(1, 0, 2)
    kt = torch.from_numpy(k).double().permute(1, 0, 2)
    vt = torch.from_numpy(v).double().permute(1, 0, 2)
    G = qt.shape[0] // kt.shape[0]
    kt = kt.repeat_interleave(G, dim=0)  # consecutive q-heads share a kv-head
    vt = vt.repeat_interleave(G, dim=0)
    o = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, attn_mask=mask, is_causal=causal, scale=scale)
    return o.permute(1, 0, 2).numpy()


def test_full_causal_equals_library_sdpa_with_gqa_and_scale():
    L, Hq, Hkv, D = 77, 6, 2, 32
    q, k, v = _bf16_randn((L, Hq, D), 10), _bf16_randn((L, Hkv, D), 11), _bf16_randn((L, Hkv, D), 12)
    for scale in (None, 0.37):
        got = oracle.prefill(q, k, v, [0, L], 1, 0, True, scale=scale)
        want = _sdpa_f64(q, k, v, causal=True, scale=scale)
        np.testing.assert_allclose(got["out"], want, rtol=1e-12, atol=1e-13)
        np.testing.assert_allclose(got["psum"], 1.0, atol=1e-12)
        assert (got["nvis"][:, 0] == np.arange(1, L + 1)).all()


def test_window_covering_context_is_full_attention():
    """Sec. 4.1.2: SWA is identical to full attention when the context fits the window."""
    L, Hq, Hkv, D = 50, 4, 2, 16
    q, k, v = _bf16_randn((L, Hq, D), 20), _bf16_randn((L, Hkv, D), 21), _bf16_randn((L, Hkv, D), 22)
    full = oracle.prefill(q, k, v, [0, L], 1, 0, True)
    for W, S in ((L, 0), (L + 5, 3), (10 * L, 0)):
        swa = oracle.prefill(q, k, v, [0, L], W, S, False)
        assert np.array_equal(swa["out"], full["out"])
        assert np.array_equal(swa["lse"], full["lse"])
    almost = oracle.prefill(q, k, v, [0, L], L - 1, 0, False)  # one key short on the last row only
    assert np.array_equal(almost["out"][:-1], full["out"][:-1])
    assert not np.array_equal(almost["out"][-1], full["out"][-1])


def test_banded_mask_equals_library_sdpa_with_band_matrix():
    """SWA + sinks against the library routine fed a band built from tril diagonals."""
    L, Hq, Hkv, D = 90, 4, 4, 32
    q, k, v = _bf16_randn((L, Hq, D), 30), _bf16_randn((L, Hkv, D), 31), _bf16_randn((L, Hkv, D), 32)
    ones = torch.ones(L, L, dtype=torch.bool)
    for W, S in ((1, 0), (7, 0), (16, 3), (5, 9), (33, 40)):
        band = torch.tril(ones) & ~torch.tril(ones, diagonal=-W)  # W diagonals: 0, -1, ..., -(W-1)
        sink = torch.tril(ones).clone()
        sink[:, S:] = False
        got = oracle.prefill(q, k, v, [0, L], W, S, False)
        want = _sdpa_f64(q, k, v, mask=band | sink)
        np.testing.assert_allclose(got["out"], want, rtol=1e-12, atol=1e-13)
        assert (got["nvis"][:, 0] == (band | sink).sum(1).numpy()).all()


def test_window_one_no_sink_returns_own_value():
    L, Hq, Hkv, D = 40, 4, 2, 8
    q, k, v = _bf16_randn((L, Hq, D), 40), _bf16_randn((L, Hkv, D), 41), _bf16_randn((L, Hkv, D), 42)
    got = oracle.prefill(q, k, v, [0, L], 1, 0, False)
    want = np.repeat(v.astype(np.float64), Hq // Hkv, axis=1)  # q-head h reads kv-head h // G
    assert np.array_equal(got["out"], want)
    assert (got["nvis"] == 1).all()


def test_zero_query_gives_mean_of_visible_values_and_log_count():
    L, Hq, Hkv, D, W, S = 60, 2, 1, 8, 9, 3
    q = np.zeros((L, Hq, D), np.float32)
    k, v = _bf16_randn((L, Hkv, D), 51), _bf16_randn((L, Hkv, D), 52)
    got = oracle.prefill(q, k, v, [0, L], W, S, False)
    for i in range(L):
        vis = sorted(_range_union_visible(i, W, S, False))
        np.testing.assert_allclose(got["out"][i, 0], v[vis, 0].astype(np.float64).mean(0), rtol=1e-13, atol=1e-14)
        np.testing.assert_allclose(got["lse"][i, 0], np.log(len(vis)), rtol=1e-13)


def test_probabilities_sum_to_one_and_bruteforce_rows():
    """Every row: softmax written out by hand in numpy over the range-union key set."""
    L, Hq, Hkv, D = 45, 4, 2, 16
    q, k, v = _bf16_randn((L, Hq, D), 60), _bf16_randn((L, Hkv, D), 61), _bf16_randn((L, Hkv, D), 62)
    for W, S, full in ((6, 2, False), (1, 5, False), (13, 0, False), (1, 0, True)):
        got = oracle.prefill(q, k, v, [0, L], W, S, full)
        np.testing.assert_allclose(got["psum"], 1.0, atol=1e-12)
        for i in range(L):
            vis = sorted(_range_union_visible(i, W, S, full))
            for h in range(Hq):
                s = (k[vis, h // 2].astype(np.float64) @ q[i, h].astype(np.float64)) / np.sqrt(D)
                w = np.exp(s - s.max())
                w /= w.sum()
                np.testing.assert_allclose(got["out"][i, h], w @ v[vis, h // 2].astype(np.float64),
                                           rtol=1e-11, atol=1e-13)
                np.testing.assert_allclose(got["lse"][i, h], np.log(np.exp(s).sum()), rtol=1e-12)


def test_packed_sequences_are_independent_and_sinks_are_per_sequence():
    lens, Hq, Hkv, D, W, S = (9, 1, 30, 17), 4, 2, 16, 5, 2
    T = sum(lens)
    q, k, v = _bf16_randn((T, Hq, D), 70), _bf16_randn((T, Hkv, D), 71), _bf16_randn((T, Hkv, D), 72)
    cu = np.concatenate([[0], np.cumsum(lens)])
    packed = oracle.prefill(q, k, v, cu, W, S, False)
    for b, n in enumerate(lens):
        a, e = cu[b], cu[b + 1]
        alone = oracle.prefill(q[a:e], k[a:e], v[a:e], [0, n], W, S, False)
        assert np.array_equal(packed["out"][a:e], alone["out"])
        assert np.array_equal(packed["nvis"][a:e], alone["nvis"])


def test_row_selection_matches_full_run():
    L, Hq, Hkv, D = 64, 4, 2, 8
    q, k, v = _bf16_randn((L, Hq, D), 80), _bf16_randn((L, Hkv, D), 81), _bf16_randn((L, Hkv, D), 82)
    allrows = oracle.prefill(q, k, v, [0, 20, L], 7, 1, False)
    rt, rh = np.array([0, 19, 20, 63, 33]), np.array([0, 3, 1, 2, 0])
    some = oracle.prefill(q, k, v, [0, 20, L], 7, 1, False, rows=(rt, rh))
    assert np.array_equal(some["out"], allrows["out"][rt, rh])
    assert np.array_equal(some["lse"], allrows["lse"][rt, rh])


def test_large_fixture_count_through_nvis():
    """L=32768, W=2048, S=4 (the long-context workload): per-row visible counts sum to the closed form."""
    L, W, S = 32768, 2048, 4
    rt = np.arange(L)
    z = np.zeros((L, 1, 1), np.float32)
    got = oracle.prefill(z, z, z, [0, L], W, S, False, rows=(rt, np.zeros(L, np.int32)))
    assert int(got["nvis"].sum()) == 65135610
    np.testing.assert_allclose(got["lse"], np.log(got["nvis"]), rtol=1e-12)


def test_decode_is_last_prefill_row():
    """Sec. 3.1.1: the generated token sees the whole context (is_full) or window+sinks (SWA decode)."""
    B, Lmax, Hq, Hkv, D = 3, 70, 4, 2, 16
    q = _bf16_randn((B, Hq, D), 90)
    kc, vc = _bf16_randn((B, Lmax, Hkv, D), 91), _bf16_randn((B, Lmax, Hkv, D), 92)
    seqlens = [70, 1, 37]
    for W, S, full in ((8, 2, False), (1, 0, False), (100, 0, False), (1, 0, True)):
        got = oracle.decode(q, kc, vc, seqlens, W, S, full)
        for b, n in enumerate(seqlens):
            qq = np.zeros((n, Hq, D), np.float32)
            qq[n - 1] = q[b]
            ref = oracle.prefill(qq, kc[b, :n], vc[b, :n], [0, n], W, S, full)
            assert np.array_equal(got["out"][b], ref["out"][n - 1])
            want_n = n if full else len(_range_union_visible(n - 1, W, S, False))
            assert (got["nvis"][b] == want_n).all()
    # library check for FA decode: softmax over all valid entries
    got = oracle.decode(q, kc, vc, seqlens, 1, 0, True)
    for b, n in enumerate(seqlens):
        for h in range(Hq):
            s = torch.from_numpy(kc[b, :n, h // 2]).double() @ torch.from_numpy(q[b, h]).double() / np.sqrt(D)
            want = torch.softmax(s, 0) @ torch.from_numpy(vc[b, :n, h // 2]).double()
            np.testing.assert_allclose(got["out"][b, h], want.numpy(), rtol=1e-12, atol=1e-13)


def test_split_partition_invariance_of_the_definition():
    """Any partition of the visible keys recombined by log-sum-exp gives the unsplit result (what a
    split-K decode relies on).  The partial results come from the oracle run on key subsets via is_full
    on truncated/rolled caches; the recombination is written out here."""
    Lmax, Hq, Hkv, D = 64, 2, 1, 8
    q = _bf16_randn((1, Hq, D), 100)
    kc, vc = _bf16_randn((1, Lmax, Hkv, D), 101), _bf16_randn((1, Lmax, Hkv, D), 102)
    whole = oracle.decode(q, kc, vc, [Lmax], 1, 0, True)
    for cuts in ([0, 64], [0, 1, 64], [0, 9, 10, 33, 64], [0, 32, 64]):
        parts = []
        for a, e in zip(cuts[:-1], cuts[1:]):
            r = oracle.decode(q, kc[:, a:e], vc[:, a:e], [e - a], 1, 0, True)
            parts.append((r["lse"][0], r["out"][0]))
        M = np.max([p[0] for p in parts], axis=0)
        den = sum(np.exp(p[0] - M) for p in parts)
        num = sum(np.exp(p[0] - M)[:, None] * p[1] for p in parts)
        np.testing.assert_allclose(num / den[:, None], whole["out"][0], rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(M + np.log(den), whole["lse"][0], rtol=1e-12)


def test_layer_schedule_patterns_from_the_paper():
    with open(os.path.join(GOLDEN, "fa_layer_patterns.txt")) as f:
        rows = [ln for ln in f if ln.strip() and not ln.startswith("#")]
    for ln in rows:
        name, start, step, first, count = [x.strip() for x in ln.split(";")]
        start, step, count = int(start), int(step), int(count)
        fa = [l for l in range(36) if oracle.layer_is_full(l, start, step, False, 0)]
        assert len(fa) == count, name
        want_first = [int(x) for x in first.split()]
        assert fa[: len(want_first)] == want_first, name
        # FA layers are full in both phases; FA decode makes every layer full while decoding only
        assert [l for l in range(36) if oracle.layer_is_full(l, start, step, False, 1)] == fa
        assert all(oracle.layer_is_full(l, start, step, True, 1) for l in range(36))
        assert [l for l in range(36) if oracle.layer_is_full(l, start, step, True, 0)] == fa


def test_planted_mistakes_would_be_caught():
    """Sanity of the pins themselves: the range-union statement with a W+1 window, or without the sink
    clamp to the causal prefix, differs from the oracle on this grid."""
    def wrong_window(i, W, S):
        return set(range(max(0, i - W), i + 1)) | set(range(0, min(S, i + 1)))

    def sinks_not_causal(i, W, S):
        return set(range(max(0, i - W + 1), i + 1)) | set(range(0, S))

    for wrong in (wrong_window, sinks_not_causal):
        differs = False
        for L, W, S in GRID:
            for i in range(L):
                got = {j for j in range(L) if oracle.visible(i, j, W, S, False)}
                if got != {j for j in wrong(i, W, S) if j < L}:
                    differs = True
        assert differs

"""Pins for the oracle functions behind the multi-device forms of the path (CPU only): decode with the cache cut
along the context (partial results + log-sum-exp combine), context-parallel prefill (halo + sink rows), the
per-sequence mask policy of a mixed batch, and the explicit FA-layer set with its selection by lazy ratio.

What could go wrong and which test catches it: the mask evaluated on shard-local instead of absolute positions
(partition test with sinks and a window that straddles shard borders), a shard's maximum taken over invisible
keys or the combine weights inverted (hand-computed two-key case, partition invariance), an empty shard poisoning
the result (empty-shard cases), the halo offset applied with the wrong sign or the sink rows read for positions
that are local (chunks-with-halo reproduce the one-shot prefill bit for bit, rank 0 with key_pos0 = 0), a halo
that is too short accepted silently (raises), ties and the lazy / non-lazy orientation in the layer selection.
"""
import numpy as np
import pytest
import torch

import oracle


def _bf16_randn(shape, seed):
    g = torch.Generator().manual_seed(seed)
    return torch.randn(shape, generator=g).to(torch.bfloat16).to(torch.float32).numpy()


# ------------------------------------------------------------------------------------------ split-KV decode
def test_partial_of_two_keys_by_hand():
    """One head, D = 2, a shard holding positions 5 and 6 of a 7-token sequence, scale 1."""
    q = np.array([[[1.0, 2.0]]], dtype=np.float32)
    ks = np.array([[[[0.5, 0.25]], [[-1.0, 1.0]]]], dtype=np.float32)   # scores 1.0 and 1.0
    vs = np.array([[[[2.0, 0.0]], [[0.0, 4.0]]]], dtype=np.float32)
    r = oracle.decode_partial(q, ks, vs, [7], 5, 100, 0, False, scale=1.0)
    assert np.allclose(r["part"][0, 0], [1.0, 2.0, 2.0, 4.0], atol=1e-15) and r["nvis"][0, 0] == 2
    # window of one key: only position 6 is visible
    r = oracle.decode_partial(q, ks, vs, [7], 5, 1, 0, False, scale=1.0)
    assert np.allclose(r["part"][0, 0], [1.0, 1.0, 0.0, 4.0], atol=1e-15) and r["nvis"][0, 0] == 1
    # the same shard claimed to sit at positions 0, 1 with a window of one: nothing visible, the empty partial
    r = oracle.decode_partial(q, ks, vs, [7], 0, 1, 0, False, scale=1.0)
    assert r["part"][0, 0, 0] == -np.inf and (r["part"][0, 0, 1:] == 0).all() and r["nvis"][0, 0] == 0
    # ... but with two sink tokens both are visible again
    r = oracle.decode_partial(q, ks, vs, [7], 0, 1, 2, False, scale=1.0)
    assert r["nvis"][0, 0] == 2


def test_combine_by_hand():
    """Two partials of one row: (m=0, l=1, o=[2]) and (m=ln 3, l=2, o=[8]) -> (1*2 + 3*8) / (1*1 + 3*2) = 26/7;
    an empty partial in between changes nothing."""
    empty = [-np.inf, 0.0, 0.0]
    parts = np.array([[[[0.0, 1.0, 2.0]]], [[empty]], [[[np.log(3.0), 2.0, 8.0]]]])
    assert np.allclose(oracle.decode_combine(parts), 26.0 / 7.0, atol=1e-14)
    assert (oracle.decode_combine(np.array([[[empty]]])) == 0).all()


@pytest.mark.parametrize("W,S,full", [(9, 3, False), (40, 0, False), (1, 0, True), (5, 30, False)])
@pytest.mark.parametrize("cuts", [(0, 64), (0, 32, 64), (0, 7, 8, 8, 50, 64), (0, 1, 63, 64)])
def test_decode_is_invariant_under_any_partition_of_the_cache(W, S, full, cuts):
    B, Lmax, Hq, Hkv, D = 3, 64, 4, 2, 16
    sl = [64, 10, 33]          # the shorter sequences leave whole shards without a valid entry
    q = _bf16_randn((B, Hq, D), 200)
    kc, vc = _bf16_randn((B, Lmax, Hkv, D), 201), _bf16_randn((B, Lmax, Hkv, D), 202)
    kc[1, 10:] = np.nan        # entries past a sequence's length are never visible, whatever they hold
    vc[1, 10:] = np.nan
    want = oracle.decode(q, np.nan_to_num(kc), np.nan_to_num(vc), sl, W, S, full)
    parts, seen = [], 0
    for a, b in zip(cuts[:-1], cuts[1:]):
        r = oracle.decode_partial(q, kc[:, a:b], vc[:, a:b], sl, a, W, S, full)
        parts.append(r["part"])
        seen = seen + r["nvis"]
    got = oracle.decode_combine(np.stack(parts))
    assert np.allclose(got, want["out"], rtol=0, atol=1e-13)
    assert np.array_equal(seen, want["nvis"])
    # one shard holding everything: the partial is the unnormalised answer and its log-sum-exp
    whole = oracle.decode_partial(q, kc, vc, sl, 0, W, S, full)["part"]
    assert np.allclose(whole[..., 2:] / whole[..., 1:2], want["out"], rtol=0, atol=1e-13)
    assert np.allclose(whole[..., 0] + np.log(whole[..., 1]), want["lse"], rtol=0, atol=1e-13)


# ------------------------------------------------------------------------------------ context-parallel prefill
@pytest.mark.parametrize("W,S", [(16, 3), (7, 0), (5, 12), (200, 2)])
@pytest.mark.parametrize("P", [2, 3, 5])
def test_stretches_with_halo_and_sink_rows_reproduce_the_one_shot_prefill(W, S, P):
    """Each of P participants owns a contiguous stretch of both sequences, gets the W - 1 keys before it as a halo
    and the first S keys as sink rows: its rows are, bit for bit, those of the self-attention prefill."""
    lens, Hq, Hkv, D = [90, 47], 4, 2, 16
    cu = np.concatenate([[0], np.cumsum(lens)])
    T = cu[-1]
    q, k, v = _bf16_randn((T, Hq, D), 210), _bf16_randn((T, Hkv, D), 211), _bf16_randn((T, Hkv, D), 212)
    whole = oracle.prefill(q, k, v, cu, W, S, False)
    sink_rows = max(S, 1)
    sk = np.stack([np.pad(k[cu[b]:cu[b] + sink_rows], ((0, max(0, sink_rows - lens[b])), (0, 0), (0, 0))) for b in range(2)])
    sv = np.stack([np.pad(v[cu[b]:cu[b] + sink_rows], ((0, max(0, sink_rows - lens[b])), (0, 0), (0, 0))) for b in range(2)])
    for r in range(P):
        qs, ks, vs, lq, lk, p0, rows = [], [], [], [], [], [], []
        for b, n in enumerate(lens):
            own0, own1 = n * r // P, n * (r + 1) // P
            h0 = max(0, own0 - (W - 1))
            qs.append(q[cu[b] + own0:cu[b] + own1]); ks.append(k[cu[b] + h0:cu[b] + own1]); vs.append(v[cu[b] + h0:cu[b] + own1])
            lq.append(own1 - own0); lk.append(own1 - h0); p0.append(h0)
            rows.append(np.arange(cu[b] + own0, cu[b] + own1))
        got = oracle.prefill_cp(np.concatenate(qs), np.concatenate(ks), np.concatenate(vs), sk, sv,
                                np.concatenate([[0], np.cumsum(lq)]), np.concatenate([[0], np.cumsum(lk)]), p0, W, S, False)
        rows = np.concatenate(rows)
        assert np.array_equal(got["out"], whole["out"][rows])
        assert np.array_equal(got["lse"], whole["lse"][rows])
        assert np.array_equal(got["nvis"], whole["nvis"][rows])


def test_context_parallel_reduces_to_chunked_prefill_and_rejects_a_short_halo():
    lq, lk, Hq, Hkv, D, W, S = 9, 30, 4, 2, 16, 8, 2
    q, k, v = _bf16_randn((lq, Hq, D), 220), _bf16_randn((lk, Hkv, D), 221), _bf16_randn((lk, Hkv, D), 222)
    none = np.zeros((1, 0, Hkv, D), dtype=np.float32)
    a = oracle.prefill_cp(q, k, v, none, none, [0, lq], [0, lk], [0], W, S, False)
    b = oracle.prefill_chunked(q, k, v, [0, lq], [0, lk], W, S, False)
    assert np.array_equal(a["out"], b["out"])
    # local keys start at position 25 of a longer context: queries at 46..54 need keys from 39 on: enough halo ...
    sink = _bf16_randn((1, S, Hkv, D), 223)
    oracle.prefill_cp(q, k, v, sink, sink, [0, lq], [0, lk], [25], W, S, False)
    # ... but a window of 30 reaches back to position 17 < 25, and full attention needs everything
    with pytest.raises(ValueError):
        oracle.prefill_cp(q, k, v, sink, sink, [0, lq], [0, lk], [25], 30, S, False)
    with pytest.raises(ValueError):
        oracle.prefill_cp(q, k, v, sink, sink, [0, lq], [0, lk], [25], W, S, True)
    # and missing sink rows are noticed too
    with pytest.raises(ValueError):
        oracle.prefill_cp(q, k, v, none, none, [0, lq], [0, lk], [25], W, S, False)


# --------------------------------------------------------------------------------------- mixed batch
def test_per_sequence_policy_equals_per_sequence_calls():
    Hq, Hkv, D, W, S = 4, 2, 16, 6, 2
    lq, lk, fs = [4, 1, 9, 1], [10, 40, 9, 25], [0, 1, 0, 1]   # prefill chunks under SWA next to decode tokens under FA
    qs = [_bf16_randn((n, Hq, D), 230 + i) for i, n in enumerate(lq)]
    ks = [_bf16_randn((n, Hkv, D), 240 + i) for i, n in enumerate(lk)]
    vs = [_bf16_randn((n, Hkv, D), 250 + i) for i, n in enumerate(lk)]
    cq, ck = np.concatenate([[0], np.cumsum(lq)]), np.concatenate([[0], np.cumsum(lk)])
    mixed = oracle.prefill_chunked(np.concatenate(qs), np.concatenate(ks), np.concatenate(vs), cq, ck, W, S, False,
                                   is_full_seq=fs)
    for b in range(4):
        alone = oracle.prefill_chunked(qs[b], ks[b], vs[b], [0, lq[b]], [0, lk[b]], W, S, bool(fs[b]))
        assert np.array_equal(mixed["out"][cq[b]:cq[b + 1]], alone["out"])
        assert np.array_equal(mixed["nvis"][cq[b]:cq[b + 1]], alone["nvis"])
    # first query of sequence 0 sits at position 6: window keys 1..6 and sink keys 0, 1 -> 7 keys (key 1 counted once)
    assert (mixed["nvis"][cq[1]] == 40).all() and (mixed["nvis"][cq[0]] == 7).all()
    # the flags, not the scalar, decide
    again = oracle.prefill_chunked(np.concatenate(qs), np.concatenate(ks), np.concatenate(vs), cq, ck, W, S, True,
                                   is_full_seq=fs)
    assert np.array_equal(again["out"], mixed["out"])


# --------------------------------------------------------------------------------------- layer sets
def test_explicit_fa_layer_set_and_the_printed_patterns():
    """An explicit set reproduces every fixed-interval pattern of Table 1, and FA decode overrides it in the decode
    phase only."""
    for start, step in ((1, 2), (0, 2), (1, 4), (1, 8), (3, 4)):
        mask = np.zeros(36, dtype=np.uint8)
        mask[start::step] = 1
        for l in range(36):
            for phase in (0, 1):
                for fa_decode in (False, True):
                    assert oracle.layer_is_full_mask(l, mask, fa_decode, phase) == \
                        oracle.layer_is_full(l, start, step, fa_decode, phase)
    odd = np.array([0, 1, 1, 0, 0, 0, 1], dtype=np.uint8)   # not periodic
    assert [oracle.layer_is_full_mask(l, odd, False, 0) for l in range(7)] == [bool(x) for x in odd]
    assert all(oracle.layer_is_full_mask(l, odd, True, 1) for l in range(7))


def test_selection_by_lazy_ratio():
    """"lazy" = the half of the layers with the higher ratio; FA goes to the non-lazy half (the method as proposed)
    or to the lazy half (the variant of the paper's LightTransfer table)."""
    ratio = [0.9, 0.1, 0.5, 0.7, 0.3, 0.8]
    assert oracle.select_fa_layers(ratio, 3, False).tolist() == [0, 1, 1, 0, 1, 0]
    assert oracle.select_fa_layers(ratio, 3, True).tolist() == [1, 0, 0, 1, 0, 1]
    # against a sort, on random ratios; the two orientations are complements; sizes are exact
    rng = np.random.default_rng(3)
    for n, n_lazy in ((36, 18), (36, 27), (5, 0), (5, 5), (1, 1)):
        r = rng.random(n)
        lazy = set(np.argsort(-r, kind="stable")[:n_lazy].tolist())
        on_lazy = oracle.select_fa_layers(r, n_lazy, True)
        assert set(np.nonzero(on_lazy)[0].tolist()) == lazy
        assert np.array_equal(oracle.select_fa_layers(r, n_lazy, False), 1 - on_lazy)
    # ties: the lower index counts as the lazier
    assert oracle.select_fa_layers([0.5, 0.5, 0.5, 0.5], 2, True).tolist() == [1, 1, 0, 0]
    with pytest.raises(ValueError):
        oracle.select_fa_layers([0.1, 0.2], 3, True)

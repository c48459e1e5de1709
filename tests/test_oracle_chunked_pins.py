"""Pins for the chunked-prefill oracle (queries = the last len_q tokens of a len_k-token context).  CPU only.

What could go wrong and which test catches it: the position offset len_k - len_q dropped or applied with
the wrong sign (numpy brute force, decode equivalence), keys taken from the wrong sequence of the
packed key buffer (packed-batch test), sinks or window measured from the chunk instead of the
sequence (numpy brute force with W and S smaller than the offset).
"""
import numpy as np
import pytest
import torch

import oracle


def _bf16_randn(shape, seed):
    g = torch.Generator().manual_seed(seed)
    return torch.randn(shape, generator=g).to(torch.bfloat16).to(torch.float32).numpy()


def _visible_positions(pos, W, S, is_full):
    """Keys a query at position `pos` sees, as a union of index ranges (window of W keys ending at the
    query AND the first S tokens; Sec. 3.2.1), not as the oracle's predicate."""
    if is_full:
        return list(range(pos + 1))
    return sorted(set(range(max(0, pos - W + 1), pos + 1)) | set(range(min(S, pos + 1))))


def _numpy_rows(q, k, v, lq, lk, W, S, is_full, scale):
    """Hand-written float64 softmax over the range-union key set, one sequence."""
    Hq, Hkv = q.shape[1], k.shape[1]
    G = Hq // Hkv
    out = np.zeros((lq, Hq, q.shape[2]))
    for i in range(lq):
        keys = _visible_positions(lk - lq + i, W, S, is_full)
        for h in range(Hq):
            s = (k[keys, h // G].astype(np.float64) @ q[i, h].astype(np.float64)) * scale
            p = np.exp(s - s.max())
            out[i, h] = (p / p.sum()) @ v[keys, h // G].astype(np.float64)
    return out


@pytest.mark.parametrize("lq,lk", [(1, 1), (5, 5), (3, 40), (17, 64), (40, 41)])
@pytest.mark.parametrize("W,S,full", [(1, 0, False), (8, 0, False), (8, 3, False), (5, 20, False), (100, 0, False), (1, 0, True)])
def test_chunked_matches_numpy_bruteforce(lq, lk, W, S, full):
    Hq, Hkv, D = 4, 2, 16
    q, k, v = _bf16_randn((lq, Hq, D), 1), _bf16_randn((lk, Hkv, D), 2), _bf16_randn((lk, Hkv, D), 3)
    r = oracle.prefill_chunked(q, k, v, [0, lq], [0, lk], W, S, full, scale=0.3)
    want = _numpy_rows(q, k, v, lq, lk, W, S, full, 0.3)
    assert np.allclose(r["out"], want, rtol=0, atol=1e-12)
    assert np.allclose(r["psum"], 1.0, atol=1e-12)
    for i in range(lq):
        assert (r["nvis"][i] == len(_visible_positions(lk - lq + i, W, S, full))).all()


def test_chunks_reproduce_the_one_shot_prefill():
    """Feeding a prompt in chunks (each chunk's queries against the context so far) gives the rows of the
    self-attention prefill of the whole prompt (Fig. 1a: later tokens attend to the stored context)."""
    L, Hq, Hkv, D, W, S = 90, 4, 2, 16, 16, 3
    q, k, v = _bf16_randn((L, Hq, D), 4), _bf16_randn((L, Hkv, D), 5), _bf16_randn((L, Hkv, D), 6)
    whole = oracle.prefill(q, k, v, [0, L], W, S, False)
    done = 0
    for chunk in (7, 32, 1, 50):
        end = done + chunk
        r = oracle.prefill_chunked(q[done:end], k[:end], v[:end], [0, chunk], [0, end], W, S, False)
        assert np.array_equal(r["out"], whole["out"][done:end])
        assert np.array_equal(r["nvis"], whole["nvis"][done:end])
        done = end
    assert done == L


def test_chunk_of_one_token_is_decode():
    B, Lmax, Hq, Hkv, D = 3, 50, 4, 2, 16
    sl = [50, 1, 23]
    q = _bf16_randn((B, Hq, D), 7)
    kc, vc = _bf16_randn((B, Lmax, Hkv, D), 8), _bf16_randn((B, Lmax, Hkv, D), 9)
    kp = np.concatenate([kc[b, :n] for b, n in enumerate(sl)])
    vp = np.concatenate([vc[b, :n] for b, n in enumerate(sl)])
    cu_k = np.concatenate([[0], np.cumsum(sl)])
    for W, S, full in ((8, 2, False), (1, 0, True)):
        a = oracle.prefill_chunked(q, kp, vp, np.arange(B + 1), cu_k, W, S, full)
        b = oracle.decode(q, kc, vc, sl, W, S, full)
        assert np.array_equal(a["out"], b["out"])


def test_packed_batch_sequences_are_independent_and_equal_lengths_reduce_to_prefill():
    Hq, Hkv, D, W, S = 4, 2, 16, 6, 2
    lq, lk = [4, 9, 1], [10, 9, 30]
    qs = [_bf16_randn((n, Hq, D), 10 + i) for i, n in enumerate(lq)]
    ks = [_bf16_randn((n, Hkv, D), 20 + i) for i, n in enumerate(lk)]
    vs = [_bf16_randn((n, Hkv, D), 30 + i) for i, n in enumerate(lk)]
    cq, ck = np.concatenate([[0], np.cumsum(lq)]), np.concatenate([[0], np.cumsum(lk)])
    packed = oracle.prefill_chunked(np.concatenate(qs), np.concatenate(ks), np.concatenate(vs), cq, ck, W, S, False)
    for b in range(3):
        alone = oracle.prefill_chunked(qs[b], ks[b], vs[b], [0, lq[b]], [0, lk[b]], W, S, False)
        assert np.array_equal(packed["out"][cq[b]:cq[b + 1]], alone["out"])
    # len_q == len_k everywhere: the self-attention prefill
    same = oracle.prefill_chunked(np.concatenate(ks).repeat(2, axis=1), np.concatenate(ks), np.concatenate(vs), ck, ck, W, S,
                                  False)
    ref = oracle.prefill(np.concatenate(ks).repeat(2, axis=1), np.concatenate(ks), np.concatenate(vs), ck, W, S, False)
    assert np.array_equal(same["out"], ref["out"])


def test_chunked_rejects_more_queries_than_keys():
    q, k = _bf16_randn((5, 2, 8), 1), _bf16_randn((4, 2, 8), 2)
    with pytest.raises(ValueError):
        oracle.prefill_chunked(q, k, k, [0, 5], [0, 4], 4, 0, False)


def test_paged_decode_honours_the_block_table():
    """A dense cache scattered over pages in random order, unused pages and rows poisoned with NaN."""
    rng = np.random.default_rng(11)
    B, Hq, Hkv, D, page = 3, 4, 2, 16, 8
    sl = [29, 8, 1]
    max_blocks = 5
    kc, vc = _bf16_randn((B, max_blocks * page, Hkv, D), 40), _bf16_randn((B, max_blocks * page, Hkv, D), 41)
    q = _bf16_randn((B, Hq, D), 42)
    num_pages = 40
    kp = np.full((num_pages, page, Hkv, D), np.nan, dtype=np.float32)
    vp = np.full_like(kp, np.nan)
    perm = rng.permutation(num_pages)
    bt = np.full((B, max_blocks), -1, dtype=np.int32)
    nxt = 0
    for b in range(B):
        for blk in range((sl[b] + page - 1) // page):
            pg = perm[nxt]; nxt += 1
            bt[b, blk] = pg
            n = min(page, sl[b] - blk * page)
            kp[pg, :n] = kc[b, blk * page:blk * page + n]
            vp[pg, :n] = vc[b, blk * page:blk * page + n]
    for W, S, full in ((6, 2, False), (1, 0, True)):
        a = oracle.decode_paged(q, kp, vp, bt, sl, W, S, full)
        d = oracle.decode(q, kc, vc, sl, W, S, full)
        assert np.array_equal(a["out"], d["out"]) and np.isfinite(a["out"]).all()


def test_paged_prefill_honours_the_block_table():
    """The twin of the paged-decode pin for prefill_paged: packed contexts scattered over pages handed out in random
    order, unused pages and the rows past each sequence's last key poisoned with NaN.  The result must be the
    chunked prefill of the packed copy, bit for bit; a swapped j // page_size and j % page_size, a block-table row
    taken from the wrong sequence or a read past seqlens_k would surface as a mismatch or a NaN."""
    rng = np.random.default_rng(12)
    Hq, Hkv, D, page = 4, 2, 16, 8
    lq, lk = [5, 29, 1, 8], [29, 29, 17, 8]
    B, max_blocks, num_pages = len(lk), 5, 40
    ks = [_bf16_randn((n, Hkv, D), 80 + b) for b, n in enumerate(lk)]
    vs = [_bf16_randn((n, Hkv, D), 90 + b) for b, n in enumerate(lk)]
    q = _bf16_randn((sum(lq), Hq, D), 79)
    kp = np.full((num_pages, page, Hkv, D), np.nan, dtype=np.float32)
    vp = np.full_like(kp, np.nan)
    perm = rng.permutation(num_pages)
    bt = np.full((B, max_blocks), -1, dtype=np.int32)
    nxt = 0
    for b in range(B):
        for blk in range((lk[b] + page - 1) // page):
            pg = perm[nxt]; nxt += 1
            bt[b, blk] = pg
            n = min(page, lk[b] - blk * page)
            kp[pg, :n] = ks[b][blk * page:blk * page + n]
            vp[pg, :n] = vs[b][blk * page:blk * page + n]
    cq, ck = np.concatenate([[0], np.cumsum(lq)]), np.concatenate([[0], np.cumsum(lk)])
    for W, S, full in ((6, 2, False), (3, 0, False), (1, 0, True)):
        a = oracle.prefill_paged(q, kp, vp, cq, lk, bt, W, S, full)
        d = oracle.prefill_chunked(q, np.concatenate(ks), np.concatenate(vs), cq, ck, W, S, full)
        for key in ("out", "lse", "nvis"):
            assert np.array_equal(a[key], d[key]), key
        assert np.isfinite(a["out"]).all()
    rows = (np.array([0, 7, 33, 42]), np.array([3, 0, 1, 2], dtype=np.int32))
    a = oracle.prefill_paged(q, kp, vp, cq, lk, bt, 6, 2, False, rows=rows)
    d = oracle.prefill_chunked(q, np.concatenate(ks), np.concatenate(vs), cq, ck, 6, 2, False)
    assert np.array_equal(a["out"], d["out"][rows[0], rows[1]])


def test_lazy_ratio_closed_forms():
    """Q = 0 makes the softmax uniform: the share of the recent and sink keys is a count ratio.  A recent window
    that covers the whole context gives 1.  Scores that single out one old key give (almost) 0."""
    Hq, Hkv, D, lq, lk, recent, S = 4, 2, 16, 5, 40, 8, 3
    k = _bf16_randn((lk, Hkv, D), 50)
    q0 = np.zeros((lq, Hq, D), dtype=np.float32)
    r = oracle.lazy_ratio(q0, k, None, [0, lq], [0, lk], recent, S)
    want = np.mean([(recent + S) / (lk - lq + t + 1) for t in range(lq)])
    assert np.allclose(r, want, atol=1e-12)
    q = _bf16_randn((lq, Hq, D), 51)
    assert np.allclose(oracle.lazy_ratio(q, k, None, [0, lq], [0, lk], 1000, 0), 1.0, atol=1e-12)
    kk = np.zeros((lk, Hkv, D), dtype=np.float32)
    kk[10, :, 0] = 100.0  # key 10 is far outside the recent window of the last queries and not a sink
    qq = np.zeros((lq, Hq, D), dtype=np.float32)
    qq[:, :, 0] = 10.0
    assert (oracle.lazy_ratio(qq, kk, None, [0, lq], [0, lk], recent, S, scale=1.0) < 1e-300).all()


def test_lazy_ratio_equals_mass_from_two_log_sum_exps():
    """Independent route: exp(lse over recent+sink keys - lse over all keys) from the attention oracle."""
    Hq, Hkv, D, recent, S = 4, 2, 16, 6, 2
    lq, lk = [3, 4], [30, 9]
    cq, ck = np.concatenate([[0], np.cumsum(lq)]), np.concatenate([[0], np.cumsum(lk)])
    q, k = _bf16_randn((sum(lq), Hq, D), 60), _bf16_randn((sum(lk), Hkv, D), 61)
    v = _bf16_randn((sum(lk), Hkv, D), 62)
    a = oracle.prefill_chunked(q, k, v, cq, ck, recent, S, False)["lse"]
    b = oracle.prefill_chunked(q, k, v, cq, ck, 1, 0, True)["lse"]
    assert np.allclose(oracle.lazy_ratio(q, k, v, cq, ck, recent, S), np.exp(a - b).mean(axis=0), atol=1e-12)


@pytest.mark.parametrize("W,S,full", [(5, 0, False), (4, 2, False), (1, 0, True), (100, 0, False)])
def test_backward_matches_autograd_of_a_dense_masked_attention(W, S, full):
    """The analytic gradients against torch.autograd (float64) through a dense masked softmax attention built
    from a boolean mask matrix: a library routine the oracle's row formulas do not share anything with."""
    lens, Hq, Hkv, D, scale = [9, 14], 4, 2, 8, 0.37
    T = sum(lens)
    q, k, v = _bf16_randn((T, Hq, D), 70), _bf16_randn((T, Hkv, D), 71), _bf16_randn((T, Hkv, D), 72)
    dout = _bf16_randn((T, Hq, D), 73)
    cu = np.concatenate([[0], np.cumsum(lens)])
    got = oracle.prefill_backward(q, k, v, dout, cu, W, S, full, scale=scale)
    tq, tk, tv = (torch.tensor(a, dtype=torch.float64, requires_grad=True) for a in (q, k, v))
    outs = []
    for b, n in enumerate(lens):
        s0 = int(cu[b])
        i, j = torch.arange(n)[:, None], torch.arange(n)[None, :]
        mask = (j <= i) & (torch.tensor(full) | (j > i - W) | (j < S))
        kk = tk[s0:s0 + n].repeat_interleave(Hq // Hkv, dim=1)
        vv = tv[s0:s0 + n].repeat_interleave(Hq // Hkv, dim=1)
        sc = torch.einsum("ihd,jhd->hij", tq[s0:s0 + n], kk) * scale
        sc = sc.masked_fill(~mask[None], float("-inf"))
        outs.append(torch.einsum("hij,jhd->ihd", torch.softmax(sc, dim=-1), vv))
    torch.cat(outs).backward(torch.tensor(dout, dtype=torch.float64))
    fast = oracle.prefill_backward_c(q, k, v, dout, cu, W, S, full, scale=scale)
    for name, t in (("dq", tq), ("dk", tk), ("dv", tv)):
        assert np.allclose(got[name], t.grad.numpy(), rtol=0, atol=1e-11), name
        assert np.allclose(fast[name], t.grad.numpy(), rtol=0, atol=1e-11), name + " (C loops)"


@pytest.mark.parametrize("W,S,full", [(5, 0, False), (4, 2, False), (1, 0, True)])
def test_backward_rows_equals_autograd_on_the_chosen_rows_and_keys(W, S, full):
    """The row- and key-sampled gradients (used to check long sequences) against torch.autograd through a dense
    masked attention, for rows and keys that include sinks, the first and last token of each sequence and
    repeats; and against the all-rows functions."""
    lens, Hq, Hkv, D, scale = [11, 1, 17], 4, 2, 8, 0.41
    T = sum(lens)
    q, k, v = _bf16_randn((T, Hq, D), 170), _bf16_randn((T, Hkv, D), 171), _bf16_randn((T, Hkv, D), 172)
    dout = _bf16_randn((T, Hq, D), 173)
    cu = np.concatenate([[0], np.cumsum(lens)])
    tq, tk, tv = (torch.tensor(a, dtype=torch.float64, requires_grad=True) for a in (q, k, v))
    outs = []
    for b, n in enumerate(lens):
        s0 = int(cu[b])
        i, j = torch.arange(n)[:, None], torch.arange(n)[None, :]
        mask = (j <= i) & (torch.tensor(full) | (j > i - W) | (j < S))
        kk = tk[s0:s0 + n].repeat_interleave(Hq // Hkv, dim=1)
        vv = tv[s0:s0 + n].repeat_interleave(Hq // Hkv, dim=1)
        sc = torch.einsum("ihd,jhd->hij", tq[s0:s0 + n], kk) * scale
        sc = sc.masked_fill(~mask[None], float("-inf"))
        outs.append(torch.einsum("hij,jhd->ihd", torch.softmax(sc, dim=-1), vv))
    torch.cat(outs).backward(torch.tensor(dout, dtype=torch.float64))
    q_rows = (np.array([0, 10, 11, 12, 28, 5, 5]), np.array([0, 3, 1, 2, 3, 1, 1]))
    kv_rows = (np.array([0, 1, 10, 11, 12, 13, 28, 20, 20]), np.array([0, 1, 1, 0, 1, 0, 1, 0, 0]))
    got = oracle.prefill_backward_rows(q, k, v, dout, cu, W, S, full, q_rows, kv_rows, scale=scale)
    assert np.allclose(got["dq"], tq.grad.numpy()[q_rows], rtol=0, atol=1e-11)
    assert np.allclose(got["dk"], tk.grad.numpy()[kv_rows], rtol=0, atol=1e-11)
    assert np.allclose(got["dv"], tv.grad.numpy()[kv_rows], rtol=0, atol=1e-11)
    every = oracle.prefill_backward_c(q, k, v, dout, cu, W, S, full, scale=scale)
    assert np.allclose(got["dq"], every["dq"][q_rows], rtol=0, atol=1e-13)
    assert np.allclose(got["dk"], every["dk"][kv_rows], rtol=0, atol=1e-13)
    assert np.allclose(got["dv"], every["dv"][kv_rows], rtol=0, atol=1e-13)
    empty = (np.zeros(0, dtype=np.int64), np.zeros(0, dtype=np.int32))
    assert oracle.prefill_backward_rows(q, k, v, dout, cu, W, S, full, empty, empty)["dq"].shape == (0, D)
    with pytest.raises(ValueError):
        oracle.prefill_backward_rows(q, k, v, dout, cu, W, S, full, (np.array([T]), np.array([0])), empty)


def test_backward_with_a_given_forward_output():
    """The row term may be taken from a stored forward output (dout . out) instead of the probabilities.  With the
    exact output both routes are the same gradient; with a perturbed output the difference is, to first order, the
    closed form  d(dq_i) = -scale * (dout_i . e_i) * sum_j p_ij k_j,  d(dk_j) = -scale * sum_i p_ij (dout_i . e_i) q_i
    and dv does not move: this pins which tensor enters the dot product, and with which sign."""
    lens, Hq, Hkv, D, W, S, scale = [13, 6], 4, 2, 8, 5, 2, 0.33
    T = sum(lens)
    q, k, v = _bf16_randn((T, Hq, D), 180), _bf16_randn((T, Hkv, D), 181), _bf16_randn((T, Hkv, D), 182)
    dout = _bf16_randn((T, Hq, D), 183)
    cu = np.concatenate([[0], np.cumsum(lens)])
    fwd = oracle.prefill(q, k, v, cu, W, S, False, scale=scale)["out"]
    exact = oracle.prefill_backward_c(q, k, v, dout, cu, W, S, False, scale=scale)
    same = oracle.prefill_backward_c(q, k, v, dout, cu, W, S, False, scale=scale, out_given=fwd)
    for n in ("dq", "dk", "dv"):
        assert np.allclose(same[n], exact[n], rtol=0, atol=2e-6), n  # float32 copy of the exact output
    e = np.float32(1e-2) * _bf16_randn((T, Hq, D), 184)
    og = fwd.astype(np.float32) + e
    moved = oracle.prefill_backward_c(q, k, v, dout, cu, W, S, False, scale=scale, out_given=og)
    assert np.array_equal(moved["dv"], same["dv"])
    de = ((og.astype(np.float64) - fwd.astype(np.float32).astype(np.float64)) * dout).sum(-1)  # [T, Hq]
    G = Hq // Hkv
    want_dq, want_dk = np.zeros((T, Hq, D)), np.zeros((T, Hkv, D))
    for b, n in enumerate(lens):
        s0 = int(cu[b])
        for i in range(n):
            keys = np.array(_visible_positions(i, W, S, False)) + s0
            for h in range(Hq):
                sc = (k[keys, h // G].astype(np.float64) @ q[s0 + i, h].astype(np.float64)) * scale
                p = np.exp(sc - sc.max())
                p /= p.sum()
                want_dq[s0 + i, h] = -scale * de[s0 + i, h] * (p @ k[keys, h // G].astype(np.float64))
                want_dk[keys, h // G] += -scale * de[s0 + i, h] * np.outer(p, q[s0 + i, h].astype(np.float64))
    assert np.allclose(moved["dq"] - same["dq"], want_dq, rtol=0, atol=1e-12)
    assert np.allclose(moved["dk"] - same["dk"], want_dk, rtol=0, atol=1e-12)
    rows = (np.array([0, 5, 12, 13, 18]), np.array([0, 1, 2, 3, 0]))
    keys_ = (np.array([0, 1, 7, 13, 18]), np.array([0, 1, 1, 0, 1]))
    part = oracle.prefill_backward_rows(q, k, v, dout, cu, W, S, False, rows, keys_, scale=scale, out_given=og)
    assert np.allclose(part["dq"], moved["dq"][rows], rtol=0, atol=1e-13)
    assert np.allclose(part["dk"], moved["dk"][keys_], rtol=0, atol=1e-13)
    assert np.allclose(part["dv"], moved["dv"][keys_], rtol=0, atol=1e-13)

"""CPU tests of the host-side logic of the library: tile enumeration, layer schedule, symbol table.

The tile enumeration is the part of the prefill kernel that makes work linear in L (App. A); expanded to
(query, key) pairs on the CPU it must cover the oracle's visible set exactly, and tiles reported as
needing no mask must be entirely visible.
"""
import os
import re

import numpy as np
import pytest

import oracle
import paper_2512_10411_b200 as swaa
from paper_2512_10411_b200.build import build_library

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build_library()
    return swaa.load_library()


def test_library_exports_every_declared_symbol(_lib):
    with open(os.path.join(ROOT, "include", "swaa.h")) as f:
        text = f.read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = set(re.findall(r"\b(swaa_[a-z0-9_]+)\s*\(", text))
    assert {"swaa_prefill", "swaa_decode", "swaa_decode_workspace_size", "swaa_schedule_is_full",
            "swaa_schedule_fill", "swaa_status_str", "swaa_last_device_status"} <= names
    for n in sorted(names):
        assert hasattr(_lib, n), f"libswaa.so does not export {n}"


def _visible_matrix(L, W, S, full):
    return np.array([[oracle.visible(i, j, W, S, full) for j in range(L)] for i in range(L)], dtype=bool)


CASES = [(L, W, S, full) for L in (1, 5, 16, 17, 40, 67) for W in (1, 3, 8, 20, 100) for S in (0, 1, 7, 30)
         for full in (False, True) if not (full and (W, S) != (1, 0))]


@pytest.mark.parametrize("BM,BN", [(8, 8), (16, 4), (4, 16), (7, 5)])
def test_tile_enumeration_covers_exactly_the_visible_set(BM, BN):
    for L, W, S, full in CASES:
        vis = _visible_matrix(L, W, S, full)
        covered = np.zeros_like(vis)
        for m in range((L + BM - 1) // BM):
            ns, lo, hi = swaa.prefill_tile_range(L, m, BM, BN, W, S, full)
            tiles = list(range(ns)) + list(range(lo, hi + 1))
            assert len(set(tiles)) == len(tiles), "a tile is visited twice"
            i0, i1 = m * BM, min(L, (m + 1) * BM)
            for n in tiles:
                j0, j1 = n * BN, min(L, (n + 1) * BN)
                block = vis[i0:i1, j0:j1]
                assert block.any(), f"tile without a visible pair: {(L, W, S, full, m, n)}"
                if not swaa.prefill_tile_needs_mask(L, m, n, BM, BN, W, S, full):
                    assert block.all() and (n + 1) * BN <= L, (L, W, S, full, m, n)
                covered[i0:i1, j0:j1] = True
        assert not (vis & ~covered).any(), f"visible pair outside the enumerated tiles: {(L, W, S, full)}"


def test_tile_counts_of_the_benchmark_workloads():
    """Tiles visited per head at the kernel's own tile shape: linear in L for SWA, quadratic for full."""
    BM, BN = swaa.prefill_block_shape()
    assert (BM, BN) == (128, 128)

    def count(L, W, S, full):
        total = 0
        for m in range((L + BM - 1) // BM):
            ns, lo, hi = swaa.prefill_tile_range(L, m, BM, BN, W, S, full)
            total += ns + hi - lo + 1
        return total

    assert count(1024, 128, 4, False) == 21
    assert count(32768, 2048, 4, False) == 4455
    assert count(32768, 1, 0, True) == 32896
    a, b = count(32768, 2048, 4, False), count(65536, 2048, 4, False)
    assert b - a == 256 * 18  # each further query tile costs 16 band tiles + diagonal + sink tile


def test_schedule_matches_paper_patterns():
    golden = os.path.join(ROOT, "tests", "golden", "fa_layer_patterns.txt")
    with open(golden) as f:
        rows = [ln for ln in f if ln.strip() and not ln.startswith("#")]
    for ln in rows:
        name, start, step, first, count = [x.strip() for x in ln.split(";")]
        pol = swaa.SwaaPolicy(36, 2048, 10, int(start), int(step), False)
        fa = [l for l, f_ in enumerate(swaa.schedule_fill(pol, 0)) if f_]
        assert len(fa) == int(count) and fa[: len(first.split())] == [int(x) for x in first.split()], name
        for phase in (0, 1):
            for fa_decode in (False, True):
                pol = swaa.SwaaPolicy(36, 2048, 10, int(start), int(step), fa_decode)
                got = swaa.schedule_fill(pol, phase)
                want = [oracle.layer_is_full(l, int(start), int(step), fa_decode, phase) for l in range(36)]
                assert got == want
                assert [swaa.schedule_is_full(pol, l, phase) for l in range(36)] == want


def test_schedule_with_an_explicit_fa_layer_set():
    """A non-periodic FA set (what a selection by lazy ratio produces) against the oracle, in both phases."""
    rng = np.random.default_rng(8)
    for n_layers in (1, 7, 36):
        mask = rng.integers(0, 2, n_layers).tolist()
        for fa_decode in (False, True):
            pol = swaa.SwaaPolicy(n_layers, 2048, 100, 3, 4, fa_decode, fa_mask=mask)  # start / step are ignored
            for phase in (0, 1):
                want = [oracle.layer_is_full_mask(l, mask, fa_decode, phase) for l in range(n_layers)]
                assert swaa.schedule_fill(pol, phase) == want
                assert [swaa.schedule_is_full(pol, l, phase) for l in range(n_layers)] == want
    with pytest.raises(ValueError):
        swaa.schedule_fill(swaa.SwaaPolicy(4, 8, 0, 0, 0, False, fa_mask=[1, 0]), 0)


def test_fa_layers_selected_by_lazy_ratio():
    """Per-head ratios as swaa_lazy_ratio returns them -> per-layer mean -> the half with the higher ratio is "lazy";
    FA on the non-lazy half (the method as proposed) or on the lazy half (the variant of the paper's LightTransfer
    table), against the oracle's plain selection; ties, sizes and argument errors."""
    rng = np.random.default_rng(9)
    for n_layers, n_heads, n_lazy in ((36, 32, 18), (36, 8, 27), (5, 1, 0), (5, 3, 5), (1, 2, 1)):
        table = rng.random((n_layers, n_heads)).astype(np.float32)
        per_layer = table.astype(np.float64).mean(axis=1)
        for fa_on_lazy in (False, True):
            got = swaa.schedule_select_fa_layers(table, n_lazy, fa_on_lazy)
            assert got == oracle.select_fa_layers(per_layer, n_lazy, fa_on_lazy).tolist()
            assert sum(got) == (n_lazy if fa_on_lazy else n_layers - n_lazy)
            pol = swaa.SwaaPolicy(n_layers, 2048, 100, fa_decode=True, fa_mask=got)
            assert swaa.schedule_fill(pol, 0) == [bool(x) for x in got] and all(swaa.schedule_fill(pol, 1))
    assert swaa.schedule_select_fa_layers([[0.5], [0.5], [0.5], [0.5]], 2, True) == [1, 1, 0, 0]
    with pytest.raises(swaa.SwaaError):
        swaa.schedule_select_fa_layers([[0.1], [0.2]], 3, True)
    with pytest.raises(swaa.SwaaError):
        swaa.schedule_select_fa_layers([[0.1], [float("nan")]], 1, True)


def test_schedule_argument_errors():
    pol = swaa.SwaaPolicy(4, 8, 0, 1, 2, False)
    for layer, phase in ((-1, 0), (4, 0), (0, 2)):
        with pytest.raises(swaa.SwaaError):
            swaa.schedule_is_full(pol, layer, phase)
    with pytest.raises(swaa.SwaaError):
        swaa.schedule_fill(swaa.SwaaPolicy(4, 8, 0, -1, 2, False), 0)


def test_status_strings():
    assert swaa.status_str(0) == "SWAA_OK"
    assert swaa.status_str(-6) == "SWAA_ERR_TIMEOUT"
    assert swaa.status_str(-99) == "SWAA_ERR_UNKNOWN"


def test_decode_split_plan_is_consistent():
    for args in ((16, 32, 8, 128, 65536, 4096, 4, 1), (16, 32, 8, 128, 65536, 4096, 4, 0), (1, 4, 2, 64, 100, 8, 0, 0),
                 (2, 64, 4, 128, 9000, 1, 0, 1)):
        nb = swaa.decode_num_blocks(*args)
        assert nb >= 1
        B, Hq, Hkv, D = args[:4]
        heads = 8 if Hq // Hkv <= 8 else 16
        # one ticket per block and two partial slots per block, each (max, sum, O[D]) per head of a chunk
        assert swaa.decode_workspace_size(*args) >= 8 * nb + 2 * nb * heads * (D + 2) * 4
    # a problem of a single tile needs a single block
    assert swaa.decode_num_blocks(1, 4, 2, 64, 100, 8, 0, 0) == 1


def test_trimmed_cache_holds_exactly_the_visible_keys():
    """Appending tokens 0 .. len-1 into the trimmed cache leaves, in its occupied slots, exactly the positions
    the oracle's SWA predicate shows to the decode query at position len-1 (App. A)."""
    for W, S in ((1, 0), (4, 0), (4, 3), (5, 9), (16, 2), (3, 1)):
        cap = S + W
        slots = {}
        for n in range(1, 60):
            pos = n - 1
            slot = swaa.trimmed_cache_slot(pos, W, S)
            assert 0 <= slot < cap
            slots[slot] = pos
            used = swaa.trimmed_cache_len(n, W, S)
            assert used == min(n, cap) == len(slots)
            assert sorted(slots) == list(range(used))  # occupied slots are a prefix: seqlens = used addresses them
            want = {j for j in range(n) if oracle.visible(n - 1, j, W, S, False)}
            assert set(slots.values()) == want, (W, S, n)
    assert swaa.trimmed_cache_slot(-1, 4, 0) == -1 and swaa.trimmed_cache_len(5, 0, 0) == -1


def test_backward_workspace_size_covers_its_parts(_lib):
    """The backward workspace holds an fp32 dq accumulator, two fp32 row terms per (head, token) and fp32 dk/dv rows
    for the key tiles that hold sink keys (whole tiles of 128 rows, at most the packed length)."""
    size = swaa.prefill_backward_workspace_size
    B, T, Hq, Hkv, D = 3, 5000, 8, 2, 128
    base = T * Hq * D * 4 + 2 * Hq * T * 4
    assert base <= size(B, T, Hq, Hkv, D, 0) <= base + 3 * 256
    for n_sink, rows in ((1, 128), (128, 128), (129, 256), (10 ** 6, 5120)):
        want = base + 2 * B * rows * Hkv * D * 4
        assert want <= size(B, T, Hq, Hkv, D, n_sink) <= want + 3 * 256, n_sink
    assert size(0, T, Hq, Hkv, D, 4) == 256 and size(B, T, Hq, Hkv, D, -1) == 256  # invalid shapes: the minimum

"""swaa_decode_static: decode for callers that cannot allocate a workspace.

Some users of this library run attention at a point where they may not call cudaMalloc (a serving hot
path, a plug-in without access to the host framework's memory pool, a process whose device memory is
fully handed out).  For them the library carries its split-K scratch in a fixed 2 MiB array of its own.
This test calls that entry point through the C ABI twice in a row, with different shapes and masks so
that the second call finds the first call's leftovers in the shared array, and checks each result
against swaa_decode with a caller-owned workspace and against the float64 oracle.  It also watches the
driver's free-memory figure and the library's launch counter across each call: nothing may be
allocated and nothing but the one decode kernel may be launched (no clearing of the scratch).  It is
collected last on purpose.
"""
import pytest
import torch

import oracle
import paper_2512_10411_b200 as swaa
from paper_2512_10411_b200 import inputs
from helpers import ABS_TOL, REL_TOL, check_against_oracle

pytestmark = pytest.mark.gpu


def _reference(q, kc, vc, sl, W, S, full):
    B, Hq, D = q.shape
    _, Lmax, Hkv, _ = kc.shape
    ws = torch.empty(swaa.decode_workspace_size(B, Hq, Hkv, D, Lmax, W, S, full), dtype=torch.uint8, device="cuda")
    out = torch.empty_like(q)
    swaa.swaa_decode(q, kc, vc, out, sl, W, S, full, ws)
    return out


def _close(a, b):
    a, b = a.double(), b.double()
    err = (a - b).abs()
    rms = b.pow(2).mean(-1, keepdim=True).sqrt()
    return bool((err <= ABS_TOL).all() and (err <= REL_TOL * torch.maximum(b.abs(), rms)).all())


def test_decode_static_matches_decode_on_two_calls_in_a_row():
    calls = [
        # first call: sequences cut over many blocks, full attention; second: other shape, SWA mask, ragged lengths
        (inputs.DecodeConfig("a", 4, 20000, 32, 8, 128, 0, 0, seed=71, seqlens=(20000, 4101, 9000, 1)), 1, 0, True),
        (inputs.DecodeConfig("b", 3, 12000, 16, 2, 64, 0, 0, seed=72, seqlens=(12000, 5000, 300)), 4096, 4, False),
    ]
    for cfg, W, S, full in calls:
        q, kc, vc, sl = inputs.make_decode_inputs(cfg, "cuda")
        assert swaa.decode_num_blocks(cfg.B, cfg.Hq, cfg.Hkv, cfg.D, cfg.Lmax, W, S, full) > 1
        want = _reference(q, kc, vc, sl, W, S, full)
        got = torch.full_like(q, float("nan"))
        torch.cuda.synchronize()
        # torch's own counter only sees torch's allocator; the driver's free-memory figure also sees a cudaMalloc
        # made inside the library.  (The very first call in a process may load the module: it is made above, by
        # _reference, through the same kernel.)
        torch_before, free_before = torch.cuda.memory_allocated(), torch.cuda.mem_get_info()[0]
        launches_before = swaa.kernel_launch_count()
        swaa.swaa_decode_static(q, kc, vc, got, sl, W, S, full)
        assert swaa.kernel_launch_count() - launches_before == 1, "one decode kernel, no clearing launch"
        assert swaa.last_device_status() == 0
        assert torch.cuda.memory_allocated() == torch_before
        assert torch.cuda.mem_get_info()[0] >= free_before, "device memory was taken during the call"
        assert _close(got, want), cfg.name
        ref = oracle.decode(inputs.to_f32_numpy(q), inputs.to_f32_numpy(kc), inputs.to_f32_numpy(vc),
                            sl.cpu().numpy(), W, S, full)
        check_against_oracle(got, ref["out"], f"decode_static {cfg.name}")


def test_decode_static_rejects_shapes_beyond_its_scratch():
    B, Lmax, Hq, Hkv, D = 64, 65536, 64, 4, 128  # 16 query heads per kv head: the largest partial buffers
    assert swaa.decode_workspace_size(B, Hq, Hkv, D, Lmax, 1, 0, True) > swaa.DECODE_STATIC_SCRATCH_BYTES
    q = torch.zeros((B, Hq, D), dtype=torch.bfloat16, device="cuda")
    kc = torch.zeros((B, 1, Hkv, D), dtype=torch.bfloat16, device="cuda")
    # the size check comes first, so a small stand-in cache with the large Lmax claimed is never read
    lib = swaa.load_library()
    rc = lib.swaa_decode_static(q.data_ptr(), kc.data_ptr(), kc.data_ptr(), q.data_ptr(),
                                torch.ones(B, dtype=torch.int32, device="cuda").data_ptr(), B, Lmax, Hq, Hkv, D, 1, 0,
                                1, 0.0, None)
    assert rc == -4 and swaa.status_str(rc) == "SWAA_ERR_WORKSPACE"

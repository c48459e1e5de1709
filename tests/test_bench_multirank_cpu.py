"""The N > 1 path of bench.py on CPU: two gloo ranks on 127.0.0.1.  The path shards without any exchange
(every rank runs an independent replica), so all there is to test is the timing reduction (max over ranks),
the whole-job throughput, and that the reference arm prints from rank 0 only."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, os.environ["SWAA_ROOT"])
import torch.distributed as dist
import bench
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
mine = [10.0 + rank, 5.0 - rank, 1.0]            # per-rank timings: rank 1 is slower on the first, faster on the second
red = bench.max_over_ranks(mine, world)
value = bench.whole_job_value(100.0, world, red[0])
print(json.dumps({"rank": rank, "red": red, "value": value}), flush=True)
dist.destroy_process_group()
"""


SPLIT_WORKER = r"""
import os, sys, json
sys.path.insert(0, os.environ["SWAA_ROOT"])
import numpy as np, torch
import torch.distributed as dist
import bench, oracle
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
B, Lmax, Hq, Hkv, D, W, S = 3, 40, 4, 2, 8, 9, 3
g = torch.Generator().manual_seed(5)
q = torch.randn((B, Hq, D), generator=g).to(torch.bfloat16).float().numpy()
kc = torch.randn((B, Lmax, Hkv, D), generator=g).to(torch.bfloat16).float().numpy()
vc = torch.randn((B, Lmax, Hkv, D), generator=g).to(torch.bfloat16).float().numpy()
sl = [40, 7, 25]                      # rank 1 holds nothing of the second sequence
res = {}
for full in (False, True):
    a, b = Lmax * rank // world, Lmax * (rank + 1) // world
    part = oracle.decode_partial(q, kc[:, a:b], vc[:, a:b], sl, a, W, S, full)["part"]
    allp = bench.gather_decode_partials(torch.from_numpy(part), world)   # [world, B, Hq, D + 2], rank-major
    assert tuple(allp.shape) == (world, B, Hq, D + 2)
    got = oracle.decode_combine(allp.numpy())
    want = oracle.decode(q, kc, vc, sl, W, S, full)["out"]
    res[str(full)] = float(np.abs(got - want).max())
    assert np.array_equal(allp[rank].numpy(), part)   # my own partials sit in my slot (empty ones hold -inf)
print(json.dumps({"rank": rank, "err": res}), flush=True)
dist.destroy_process_group()
"""


HALO_WORKER = r"""
import os, sys, json
sys.path.insert(0, os.environ["SWAA_ROOT"])
import numpy as np, torch
import torch.distributed as dist
import bench, oracle
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
L, Hq, Hkv, D = 96, 4, 2, 8
g = torch.Generator().manual_seed(9)                       # every rank draws the same sequence and keeps its stretch
q = torch.randn((L, Hq, D), generator=g).to(torch.bfloat16).float()
k = torch.randn((L, Hkv, D), generator=g).to(torch.bfloat16).float()
v = torch.randn((L, Hkv, D), generator=g).to(torch.bfloat16).float()
own = L // world
sl = slice(rank * own, (rank + 1) * own)
res = {}
for W, S in ((17, 3), (48, 0), (5, 9)):
    kl, vl, sk, sv, p0 = bench.exchange_halo_and_sinks(k[sl].contiguous(), v[sl].contiguous(), W, S, rank, world)
    assert p0 == max(0, rank * own - (W - 1)) and kl.shape[0] == (rank + 1) * own - p0
    got = oracle.prefill_cp(q[sl].numpy(), kl.numpy(), vl.numpy(), sk.numpy(), sv.numpy(), [0, own], [0, kl.shape[0]], [p0], W, S, False)
    want = oracle.prefill(q.numpy(), k.numpy(), v.numpy(), [0, L], W, S, False)
    res[f"{W},{S}"] = bool(np.array_equal(got["out"], want["out"][sl]) and np.array_equal(got["nvis"], want["nvis"][sl]))
try:
    bench.exchange_halo_and_sinks(k[sl].contiguous(), v[sl].contiguous(), own + 2, 0, rank, world)
    res["short"] = False
except ValueError:
    res["short"] = True
print(json.dumps({"rank": rank, "ok": res}), flush=True)
dist.destroy_process_group()
"""


def _json_objects(text):
    """Every JSON object printed on stdout; two ranks that print at the same moment can end up on one line."""
    dec, out = json.JSONDecoder(), []
    for line in text.splitlines():
        i = line.find("{")
        while i >= 0:
            try:
                obj, end = dec.raw_decode(line, i)
            except json.JSONDecodeError:
                break
            out.append(obj)
            i = line.find("{", end)
    return out


def _free_port():
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        return sk.getsockname()[1]


def _launch(args, env_extra=None, timeout=300):
    env = dict(os.environ, SWAA_ROOT=ROOT, MASTER_ADDR="127.0.0.1", **(env_extra or {}))
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", str(_free_port())] + args
    return subprocess.run(cmd, capture_output=True, text=True, env=env, timeout=timeout, cwd=ROOT)


def test_two_rank_timing_reduction(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    r = _launch([str(script)])
    assert r.returncode == 0, r.stderr[-2000:]
    lines = _json_objects(r.stdout)
    assert sorted(d["rank"] for d in lines) == [0, 1]
    for d in lines:
        assert d["red"] == [11.0, 5.0, 1.0]                # element-wise max over the two ranks, on every rank
        assert d["value"] == pytest.approx(2 * 100.0 / 11.0)  # units of all ranks over the slowest rank's time


def test_reference_arm_prints_from_rank_zero_only():
    r = _launch(["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0"],
                env_extra={"OMP_NUM_THREADS": "2"}, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = _json_objects(r.stdout)
    assert len(lines) == 1
    d = lines[0]
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["cpu_baseline"]["kind"] == "oracle"
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["value"] > 0


def test_two_rank_gather_of_decode_partials(tmp_path):
    """The one exchange of a decode whose cache is cut along the context: two gloo ranks each form the partials of
    their shard (here with the oracle, on CPU), gather them through bench.gather_decode_partials and combine; every
    rank gets the result of the uncut decode."""
    script = tmp_path / "split_worker.py"
    script.write_text(SPLIT_WORKER)
    r = _launch([str(script)], env_extra={"OMP_NUM_THREADS": "2"})
    assert r.returncode == 0, r.stderr[-2000:]
    lines = _json_objects(r.stdout)
    assert sorted(d["rank"] for d in lines) == [0, 1]
    for d in lines:
        assert d["err"]["False"] < 1e-13 and d["err"]["True"] < 1e-13


def test_two_rank_halo_and_sink_exchange(tmp_path):
    """The data movement of the context-parallel prefill over two gloo ranks: after the neighbour send of the halo and
    the broadcast of the sink rows, every rank's stretch (computed with the oracle, on CPU) equals its rows of the
    one-shot prefill bit for bit; a stretch shorter than the halo is refused."""
    script = tmp_path / "halo_worker.py"
    script.write_text(HALO_WORKER)
    r = _launch([str(script)], env_extra={"OMP_NUM_THREADS": "2"})
    assert r.returncode == 0, r.stderr[-2000:]
    lines = _json_objects(r.stdout)
    assert sorted(d["rank"] for d in lines) == [0, 1]
    for d in lines:
        assert all(d["ok"].values()), d

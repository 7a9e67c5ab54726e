"""bench.py with more than one rank: the path is replicas only (no collective on the data path), so
what exists to test is the plumbing around it, run here as two gloo ranks on CPU: the max over
ranks of the timings, the whole-job aggregate, and the reference arm under torchrun (rank 0 alone
prints its line, the other rank exits 0 without work)."""
import json
import os
import socket
import subprocess
import sys
from pathlib import Path

ROOT = Path(__file__).resolve().parent.parent


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _torchrun(args, timeout=600):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port())] + args
    env = dict(os.environ, OMP_NUM_THREADS="2")
    return subprocess.run(cmd, cwd=ROOT, capture_output=True, text=True, timeout=timeout, env=env)


def test_max_over_ranks_and_aggregate_with_two_gloo_ranks(tmp_path):
    script = tmp_path / "ranks.py"
    script.write_text(
        "import os, sys, json\n"
        f"sys.path.insert(0, {str(ROOT)!r})\n"
        "import torch, torch.distributed as dist\n"
        "import bench\n"
        "dist.init_process_group('gloo')\n"
        "rank, world = dist.get_rank(), dist.get_world_size()\n"
        "ms, e2e = bench.max_over_ranks(torch, dist, [10.0 + 5.0 * rank, 30.0 - 4.0 * rank], 'cpu', world)\n"
        "out = {'rank': rank, 'ms': ms, 'e2e': e2e, 'value': bench.aggregate_value(world, 2.0e9, 4, ms)}\n"
        f"open(os.path.join({str(tmp_path)!r}, 'rank%d.json' % rank), 'w').write(json.dumps(out))\n"
        "dist.destroy_process_group()\n")
    r = _torchrun([str(script)])
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.loads((tmp_path / f"rank{i}.json").read_text()) for i in (0, 1)]
    assert sorted(l["rank"] for l in lines) == [0, 1]
    for l in lines:
        assert l["ms"] == 15.0 and l["e2e"] == 30.0                     # the slowest rank's, on every rank
        assert abs(l["value"] - 2 * 2.0e9 * 4 / 15.0e-3 / 1e9) < 1e-9     # two replicas' work in that time


def test_reference_arm_under_torchrun_prints_one_line():
    r = _torchrun(["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0"])
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.loads(l) for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    line = lines[0]
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0


def test_data_parallel_gradient_exchange_with_two_gloo_ranks(tmp_path):
    """Two CPU ranks each hold the gradients of their batch shard of a linear model; after the
    exchange every rank holds the full-batch gradient (sum) or its mean, including a parameter that
    one rank never touched."""
    script = tmp_path / "dp.py"
    script.write_text(
        "import os, sys, json\n"
        f"sys.path.insert(0, {str(ROOT)!r})\n"
        "import torch, torch.distributed as dist\n"
        "from paper_2504_06881_b200.data_parallel import all_reduce_gradients, shard_batch\n"
        "dist.init_process_group('gloo')\n"
        "rank, world = dist.get_rank(), dist.get_world_size()\n"
        "torch.manual_seed(0)\n"
        "x = torch.randn(7, 5); y = torch.randn(7, 3)\n"
        "lin = torch.nn.Linear(5, 3); extra = torch.nn.Parameter(torch.ones(4))\n"
        "full = torch.nn.functional.mse_loss(lin(x), y, reduction='sum')\n"
        "gw_full, gb_full = torch.autograd.grad(full, [lin.weight, lin.bias])\n"
        "xs, ys = shard_batch(x, rank, world), shard_batch(y, rank, world)\n"
        "loss = torch.nn.functional.mse_loss(lin(xs), ys, reduction='sum')\n"
        "if rank == 0: loss = loss + (extra * 2.0).sum()\n"
        "loss.backward()\n"
        "n = all_reduce_gradients([lin.weight, lin.bias, extra], average=False)\n"
        "ok = bool(torch.allclose(lin.weight.grad, gw_full, atol=1e-5) and torch.allclose(lin.bias.grad, gb_full, atol=1e-5)\n"
        "          and torch.allclose(extra.grad, torch.full((4,), 2.0)))\n"
        "all_reduce_gradients([lin.weight], average=True)\n"
        "ok = ok and bool(torch.allclose(lin.weight.grad, gw_full, atol=1e-5))   # equal on all ranks: the mean is itself\n"
        f"open(os.path.join({str(tmp_path)!r}, 'dp%d.json' % rank), 'w').write(json.dumps({{'ok': ok, 'n': n, 'rows': xs.shape[0]}}))\n"
        "dist.destroy_process_group()\n")
    r = _torchrun([str(script)])
    assert r.returncode == 0, r.stderr[-2000:]
    res = [json.loads((tmp_path / f"dp{k}.json").read_text()) for k in (0, 1)]
    assert all(v["ok"] for v in res) and res[0]["n"] == 15 + 3 + 4
    assert res[0]["rows"] + res[1]["rows"] == 7

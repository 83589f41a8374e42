"""The rank launcher behind `bench.py --gpus N`: two CPU ranks (gloo) started by `spawn_ranks` run
the sharded round trip with the oracle stand-in codec; both must return the single-process oracle
result, and a failing rank must surface as a non-zero exit code."""
import os
import subprocess
import sys

import numpy as np
import torch

import oracle
from paper_2405_11095_b200 import launch

HERE = os.path.dirname(os.path.abspath(__file__))


def test_rank_environment():
    env = launch.rank_environment(1, 4, 12345, base={"X": "y"})
    assert env == {"X": "y", "RANK": "1", "LOCAL_RANK": "1", "WORLD_SIZE": "4", "LOCAL_WORLD_SIZE": "4",
                   "MASTER_ADDR": "127.0.0.1", "MASTER_PORT": "12345"}
    assert 1024 < launch.free_port() < 65536


def test_two_spawned_ranks_match_the_oracle(tmp_path):
    world, M_local, d = 2, 2, 600
    cmd = [sys.executable, os.path.join(HERE, "gloo_rank_main.py"), str(tmp_path), str(M_local), str(d)]
    assert launch.spawn_ranks(cmd, world, timeout=300) == 0
    allg = torch.randn(world * M_local, d, generator=torch.Generator().manual_seed(7)).double().numpy()
    dp = oracle.padded_dim(d)
    lam = oracle.lam(float(np.linalg.norm(allg, axis=1).max()), 2.0, dp)
    lam_s = oracle.lam_server(lam, 2.0, dp)
    bits = np.stack([oracle.encode(allg[n].astype(np.float32), 5, 9, n, lam)[0] for n in range(world * M_local)])
    gbar = oracle.aggregate(bits, d, 5, 9, lam)
    res = [np.load(os.path.join(tmp_path, f"rank{r}.npz")) for r in range(world)]
    for r in res:
        np.testing.assert_allclose(r["acc"], gbar, rtol=0, atol=1e-6 * np.abs(gbar).max())
        assert (r["down"] == res[0]["down"]).all() and (r["out"] == res[0]["out"]).all()
    ref_out = oracle.downlink_decode(res[0]["down"].view(np.uint32), dp, 5, 9, lam_s)[:d]
    np.testing.assert_allclose(res[0]["out"], ref_out, rtol=0, atol=1e-5 * np.abs(ref_out).max())


def test_failing_rank_is_reported(tmp_path):
    cmd = [sys.executable, os.path.join(HERE, "gloo_rank_main.py"), str(tmp_path), "1", "100", "1"]
    assert launch.spawn_ranks(cmd, 2, timeout=300) == 3


def test_bench_spawns_ranks_itself():
    # bench.py --gpus 2 without a launcher environment goes through spawn_ranks: on this CPU machine the
    # ranks stop at the missing GPU, which shows up as a non-zero exit code of the parent and no line
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    if torch.cuda.is_available():
        return
    r = subprocess.run([sys.executable, os.path.join(os.path.dirname(HERE), "bench.py"), "--gpus", "2", "--steps", "1",
                        "--config", "0", "--no-cpu-baseline"], capture_output=True, text=True, env=env, timeout=600)
    assert r.returncode != 0 and not [x for x in r.stdout.splitlines() if x.startswith("{")]

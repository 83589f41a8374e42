"""One rank of the launcher test: started by `launch.spawn_ranks` with the rendezvous in the
environment, runs the multi-rank round trip on CPU (gloo) with the stand-in codec built on the
oracle, and writes its result to <out_dir>/rank<r>.npz."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path[:0] = [HERE, os.path.dirname(HERE)]

import oracle  # noqa: E402
from oracle_codec import OracleCodec  # noqa: E402
from paper_2405_11095_b200 import distributed as D  # noqa: E402


def main():
    out_dir, M_local, d = sys.argv[1], int(sys.argv[2]), int(sys.argv[3])
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    assert os.environ["MASTER_ADDR"] == "127.0.0.1" and int(os.environ["LOCAL_RANK"]) == rank
    dist.init_process_group("gloo")
    allg = torch.randn(world * M_local, d, generator=torch.Generator().manual_seed(7))
    grads = allg[rank * M_local:(rank + 1) * M_local]
    dp = oracle.padded_dim(d)
    lam = oracle.lam(float(allg.double().norm(dim=1).max()), 2.0, dp)
    lam_s = oracle.lam_server(lam, 2.0, dp)
    buf = D.RoundTripBuffers(bits=torch.zeros(M_local, dp // 32, dtype=torch.int32), acc=torch.zeros(dp),
                             down=torch.zeros(1, dp // 32, dtype=torch.int32), out=torch.zeros(d), ws=None)
    out = D.round_trip(OracleCodec, grads, d, buf, lam, lam_s, 5, 9, rank=rank, world=world)
    np.savez(os.path.join(out_dir, f"rank{rank}.npz"), out=out.numpy(), acc=buf.acc.numpy(), down=buf.down.numpy())
    dist.destroy_process_group()
    if len(sys.argv) > 4 and int(sys.argv[4]) == rank:
        sys.exit(3)          # the test of a failing rank


if __name__ == "__main__":
    main()

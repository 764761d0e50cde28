"""Child program of test_two_ranks_on_two_gpus_with_an_nccl_all_reduce (launched by torch.distributed.run,
one process per GPU): the worker-sharded step with the workers split over the ranks and a real NCCL
all-reduce of the packed message; rank 0 compares every rank's state with the CPU oracle.  Plain NCCL
through torch.distributed: no peer memory is handed to any kernel.  Not collected by pytest."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def main():
    from oracle import CSEROracle
    from paper_2007_13221_b200 import binding as b
    from paper_2007_13221_b200.shard import workers_of_rank
    rank, world, local = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"]), int(os.environ["LOCAL_RANK"])
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    dist.init_process_group("nccl", device_id=torch.device(dev))
    d, n, bs, R1, R2, H, eta, beta, seed, steps = 50_000 + 24, 8, 512, 4, 2, 3, 0.1, 0.9, 9, 13
    rng = np.random.default_rng(0)                       # every rank draws the same numbers
    x0 = rng.standard_normal(d).astype(np.float32)
    grads = [(rng.standard_normal(d)[None, :] + 0.5 * rng.standard_normal((n, d))).astype(np.float32)
             for _ in range(steps)]
    first, count = workers_of_rank(n, rank, world)
    opt = b.WorkerShardedCSER(d, count, n, bs, R1, R2, H, eta, beta, seed, group=dist.group.WORLD)
    opt.set_x0(torch.from_numpy(x0).to(dev))
    for g in grads:
        opt.step(torch.from_numpy(g[first:first + count]).to(dev))
    torch.cuda.synchronize()
    mine = {name: opt.state(which).cpu() for which, name in ((b.STATE_X, "x"), (b.STATE_E, "e"), (b.STATE_M, "m"))}
    gathered = [None] * world
    dist.all_gather_object(gathered, mine)
    ok = True
    if rank == 0:
        ref = CSEROracle(d, n, bs, R1, R2, H, eta, beta, seed, dtype=np.float64, exact_count=True)
        ref.set_x0(x0)
        for g in grads:
            ref.step(g)
        for name in ("x", "e", "m"):
            got = torch.cat([p[name] for p in gathered], 0).numpy().astype(np.float64)
            want = getattr(ref, name)
            rms = float(np.sqrt((want ** 2).mean()))
            bad = np.abs(got - want) > 1e-4 * np.abs(want) + 1e-4 * rms
            if bad.any():
                ok = False
                print(f"{name}: {int(bad.sum())} elements out of tolerance")
        print("WSHARD_RANKS_OK" if ok else "WSHARD_RANKS_FAILED")
    opt.close()
    dist.destroy_process_group()
    sys.exit(0 if ok else 1)


if __name__ == "__main__":
    main()

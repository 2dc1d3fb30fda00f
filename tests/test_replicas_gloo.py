"""World-size-2 check, on CPU with the gloo backend, of the host logic bench.py uses with several GPUs:
ranks draw different sequences for the same model, times are combined as the maximum over ranks, launch counts
as the sum, and the reported value is the work of all ranks over the slowest rank's time.  The path itself has
no collective (independent replicas), so nothing else crosses ranks."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    from paper_1802_00150_b200 import synth
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = synth.scaled(synth.WORKLOADS["lstm1024_b1"], I=16, H=8, steps=3)
    mine = bench.rank_workload(wl, rank)
    x = synth.inputs(mine)["x_seq"]
    w = synth.weights(wl)                 # as bench.py: the model is drawn from the un-offset workload
    # rank r "measured" 10 + r ms in total, 20 - r ms end to end, and 5 + r launches
    total, e2e, launches = bench.combine_over_ranks(dist, torch.device("cpu"), 10.0 + rank, 20.0 - rank, 5 + rank)
    value = bench.whole_job_value(world, bench.units_per_step(wl), 7, total)
    np.savez(os.path.join(out_dir, "rank%d.npz" % rank), x=x, w=w, res=np.array([total, e2e, launches, value]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_on_gloo(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    r0 = np.load(tmp_path / "rank0.npz")
    r1 = np.load(tmp_path / "rank1.npz")
    assert np.array_equal(r0["w"], r1["w"])                      # one model
    assert not np.array_equal(r0["x"], r1["x"])                  # different sequences per rank
    for r in (r0, r1):
        total, e2e, launches, value = r["res"]
        assert total == 11.0 and e2e == 20.0 and launches == 11  # MAX, MAX, SUM
        assert value == 2 * 3 * 1 * 7 / 11e-3                    # all ranks' timesteps / slowest rank's time

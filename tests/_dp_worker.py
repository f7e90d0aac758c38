"""One rank of the exact data-parallel test: runs its share of the batch and, on rank 0, saves the
weights and bit-widths after every step (run as a script by tests/test_gpu_dp.py)."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
from paper_2009_13108_b200 import Niti, NitiTrainer  # noqa: E402
from synth import config_net, make_net_inputs  # noqa: E402


def main():
    rank, world, store, out_path, cfg, batch, steps = (int(sys.argv[1]), int(sys.argv[2]), sys.argv[3], sys.argv[4],
                                                       int(sys.argv[5]), int(sys.argv[6]), int(sys.argv[7]))
    dist.init_process_group("gloo", init_method="file://" + store, rank=rank, world_size=world)
    full = config_net(cfg, batch=batch)
    x, labels, weights = make_net_inputs(full)
    share = batch // world
    net = config_net(cfg, batch=share)
    niti = Niti(0)
    tr = NitiTrainer(niti, net, weights, data_parallel=True)
    tr.load_batch(x[rank * share:(rank + 1) * share], labels[rank * share:(rank + 1) * share])
    rec = {}
    for step in range(steps):
        tr.step()
        niti.check()
        rec["hits%d" % step] = tr.global_hits().cpu().numpy()
        rec["b_fwd%d" % step] = np.array([int(b) for b in tr.b_fwd])
        rec["b_g%d" % step] = np.array([int(b) for b in tr.b_g])
        rec["b_e%d" % step] = np.array([int(b) for b in tr.b_e])
        rec["b_loss%d" % step] = np.array([int(tr.b_loss)])
        for k, w in enumerate(tr.weights):
            rec["w%d_%d" % (step, k)] = w.cpu().numpy()
    torch.cuda.synchronize()
    np.savez(out_path + ".rank%d.npz" % rank, **rec)
    dist.barrier()
    dist.destroy_process_group()
    niti.close()


if __name__ == "__main__":
    main()

"""Child process of test_dist_group_with_one_rank: ep.DistGroup (one rank per process, torch.distributed with NCCL, owner
workspace in symmetric memory, counts by all_gather, group barriers between phases) on a ONE-rank group.  With one rank
the result must be bitwise that of the plain layer; what this exercises is the orchestration a multi-GPU group runs."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))

from paper_2608_00916_b200 import ep, synth  # noqa: E402
from paper_2608_00916_b200.binding import MoELayer  # noqa: E402


def main():
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", sys.argv[1] if len(sys.argv) > 1 else "29741")
    torch.cuda.set_device(0)
    dist.init_process_group("nccl", rank=0, world_size=1)
    shape = synth.MoEShape(700, 256, 16, 4, 128)
    inp = synth.make_inputs(shape, 35)
    dev = {n: torch.from_numpy(inp[n].view(np.int16)).cuda().view(torch.bfloat16)
           for n in ("x", "W_r", "W_gate", "W_up", "W_down", "dy")}
    layer = MoELayer(shape.d, shape.E, shape.f, shape.k)
    fw = layer.forward(dev["x"], dev["W_r"], dev["W_gate"], dev["W_up"], dev["W_down"])
    bw = layer.backward(dev["dy"], 0.03)
    layer.poll()
    same = True
    for device_barrier in (True, False):
        grp = ep.DistGroup(shape.d, shape.E, shape.f, shape.k, shape.T * shape.k, device_barrier=device_barrier)
        if device_barrier:
            print("DIST_GROUP_READY", flush=True)  # the process group and the symmetric-memory rendezvous exist
            print("DEVICE_BARRIER", grp.device_barrier, flush=True)
        out = grp.forward(dev["x"], dev["W_r"], dev["W_gate"], dev["W_up"], dev["W_down"])
        sender, owner = grp.backward(dev["dy"], 0.03)
        torch.cuda.synchronize()
        grp.rk.poll()
        same = same and (torch.equal(out["y"], fw["y"]) and torch.equal(out["idx"], fw["idx"])
                         and torch.equal(sender["dx"], bw["dx"]) and torch.equal(sender["dW_r"], bw["dW_r"])
                         and all(torch.equal(owner[n], bw[n]) for n in ("dW_gate", "dW_up", "dW_down")))
        del grp
    dist.destroy_process_group()
    print("DIST_GROUP_OK" if same else "DIST_GROUP_MISMATCH")


if __name__ == "__main__":
    main()

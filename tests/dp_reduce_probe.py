"""Child process of test_grouped_reduction_through_nccl_on_a_one_rank_group: the data-parallel gradient path with the real
collective - a window of micro-batches through backward_accumulate, the last one grouped, dist.GradAllReducer reducing
every range of experts with NCCL all_reduce on its communication stream as the library signals it - on a ONE-rank NCCL
group, where the sum over the ranks is the identity: the buffers must equal those of the ungrouped, unreduced window."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))

from paper_2608_00916_b200 import dist as pdist, synth  # noqa: E402
from paper_2608_00916_b200.binding import MoELayer  # noqa: E402


def main():
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", sys.argv[1])
    torch.cuda.set_device(0)
    dist.init_process_group("nccl", rank=0, world_size=1)
    print("GROUP_READY", flush=True)
    shape = synth.MoEShape(900, 256, 16, 4, 128)
    weights = synth.make_inputs(shape, 45)
    wdev = {n: torch.from_numpy(weights[n].view(np.int16)).cuda().view(torch.bfloat16) for n in ("W_r", "W_gate", "W_up", "W_down")}
    batches = []
    for step in range(3):
        tok = synth.make_tokens(shape, 900 + step, weights["W_r"], None)
        batches.append({n: torch.from_numpy(tok[n].view(np.int16)).cuda().view(torch.bfloat16) for n in ("x", "dy")})

    def zeros():
        return {"dW_r": torch.zeros(shape.d, shape.E, device="cuda"), "dW_gate": torch.zeros(shape.E, shape.d, shape.f, device="cuda"),
                "dW_up": torch.zeros(shape.E, shape.d, shape.f, device="cuda"), "dW_down": torch.zeros(shape.E, shape.f, shape.d, device="cuda")}

    layer = MoELayer(shape.d, shape.E, shape.f, shape.k)
    ref = zeros()
    for b in batches:
        layer.forward(b["x"], wdev["W_r"], wdev["W_gate"], wdev["W_up"], wdev["W_down"])
        layer.backward_accumulate(b["dy"], 0.02, ref)
    acc = zeros()
    reducer = pdist.GradAllReducer(n_groups=4, reduce_fn=lambda t: dist.all_reduce(t, op=dist.ReduceOp.SUM, async_op=True))
    for i, b in enumerate(batches):
        layer.forward(b["x"], wdev["W_r"], wdev["W_gate"], wdev["W_up"], wdev["W_down"])
        if i + 1 < len(batches):
            layer.backward_accumulate(b["dy"], 0.02, acc)
        else:
            layer.backward_accumulate(b["dy"], 0.02, acc, group_events=reducer.events())
            reducer.start_grouped(acc)
    reducer.wait()
    torch.cuda.synchronize()
    layer.poll()
    same = all(torch.equal(acc[n], ref[n]) for n in ref)
    dist.destroy_process_group()
    print("REDUCE_OK" if same else "REDUCE_MISMATCH")


if __name__ == "__main__":
    main()

"""Worker of test_partition.py: one of two gloo ranks, each standing in for one device.

A device holds the send blocks and receive buffers of the ranks mapped to it.  Per phase it
(1) posts the blocks that cross to the other device, read from its ranks' buffers as they are at
the start of the phase, (2) performs its device-local copies, (3) stores what arrives.  The lists
come from sparbit_plan_partition_messages; the expected final state from the CPU oracle.
"""
import os
import sys
from pathlib import Path

import numpy as np
import torch
import torch.distributed as dist

sys.path.insert(0, str(Path(__file__).resolve().parent.parent))
import oracle  # noqa: E402
import paper_2109_08751_b200 as sp  # noqa: E402
import seeded_inputs as si  # noqa: E402


def main():
    mapping = sp.MAP_CYCLIC if sys.argv[1] == "cyclic" else sp.MAP_SEQUENTIAL
    me, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{os.environ['MASTER_PORT']}",
                            rank=me, world_size=world)
    other = 1 - me
    checked = 0
    for algo, P, m in ((sp.ALGO_SPARBIT, 13, 24), (sp.ALGO_SPARBIT, 16, 8), (sp.ALGO_RING, 6, 16),
                       (sp.ALGO_RECURSIVE_DOUBLING, 8, 8), (sp.ALGO_NEIGHBOR_EXCHANGE, 10, 8)):
        plan = sp.Plan(P, m, algo)
        send = si.send_blocks(P, m, seed=40 + P)
        mine = [r for r in range(P) if sp.binding.lib.sparbit_rank_device(P, world, mapping, r) == me]
        # receive buffers of this device's ranks only (dict: rank -> P slots of m bytes)
        recv = {r: np.full((P, m), si.SENTINEL, dtype=np.uint8) for r in mine}

        def src_block(msg):
            r, s = int(msg["src_rank"]), int(msg["src_slot"])
            return send[r] if int(msg["src_space"]) == sp.SPACE_SEND else recv[r][s]

        for ph in range(-1, plan.last_phase + 1):
            out = plan.partition_messages(world, mapping, ph, me, other)
            inc = plan.partition_messages(world, mapping, ph, other, me)
            loc = plan.partition_messages(world, mapping, ph, me, me)
            # (1) crossing blocks are read before anything of this phase is written
            payload = torch.from_numpy(np.stack([src_block(x) for x in out]) if len(out)
                                       else np.zeros((0, m), np.uint8))
            inbox = torch.empty((len(inc), m), dtype=torch.uint8)
            reqs = []
            if len(out):
                reqs.append(dist.isend(payload, other))
            if len(inc):
                reqs.append(dist.irecv(inbox, other))
            # (2) local copies (a phase never reads a slot it writes)
            staged = [(int(x["dst_rank"]), int(x["dst_slot"]), src_block(x).copy()) for x in loc]
            for r, s, blk in staged:
                recv[r][s] = blk
            for q in reqs:
                q.wait()
            # (3) the other device listed its blocks in the same order
            for x, blk in zip(inc, inbox.numpy()):
                recv[int(x["dst_rank"])][int(x["dst_slot"])] = blk
            dist.barrier()   # the Waitall between phases
        want, _ = oracle.allgather(algo, P, m, send)
        for r in mine:
            assert np.array_equal(recv[r].reshape(-1), want[r]), (algo, P, r)
            checked += 1
        plan.destroy()
    total = torch.tensor([checked])
    dist.all_reduce(total)
    if me == 0:
        print(f"ok {int(total)} receive buffers equal the oracle's")
    dist.destroy_process_group()


if __name__ == "__main__":
    main()

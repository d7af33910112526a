"""Worker of test_multi_device.py: one of two processes, each standing in for one device.

Both run on GPU 0 (one GPU here); on a multi-GPU node the same code runs with one GPU per process.
A process allocates the send blocks and receive buffers of its ranks, exports the receive buffers
with sparbit_ipc_export, opens the other's with sparbit_ipc_open and runs sparbit_allgather_multi.
The cross-device barrier is a stream synchronise followed by a gloo barrier: no kernel of one
process ever waits for the other.  The result is compared with the CPU oracle.
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
    me, G = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{os.environ['MASTER_PORT']}",
                            rank=me, world_size=G)
    dev = torch.device("cuda", int(os.environ.get("LOCAL_GPU", "0")) % torch.cuda.device_count())
    torch.cuda.set_device(dev)
    stream = torch.cuda.Stream(device=dev)
    opened = []
    for algo, P, m in ((sp.ALGO_SPARBIT, 13, 272), (sp.ALGO_SPARBIT, 64, 4096), (sp.ALGO_RING, 6, 48),
                       (sp.ALGO_NEIGHBOR_EXCHANGE, 10, 1024)):
        plan = sp.Plan(P, m, algo)
        host_send = si.send_blocks(P, m, seed=60 + P)
        mine = [r for r in range(P) if sp.binding.lib.sparbit_rank_device(P, G, mapping, r) == me]
        assert len(mine) == sp.multi_rank_count(P, G, mapping, me)
        send = torch.from_numpy(np.ascontiguousarray(host_send[mine]).reshape(-1)).to(dev)
        recv = torch.full((len(mine) * P * m,), si.SENTINEL, dtype=torch.uint8, device=dev)
        torch.cuda.synchronize()
        handles = [None] * G
        dist.all_gather_object(handles, sp.ipc_export(recv))
        bases = []
        for g in range(G):
            if g == me:
                bases.append(recv.data_ptr())
            else:
                ptr, base = sp.ipc_open(*handles[g])
                bases.append(ptr)
                opened.append(base)
        calls = [0]

        def barrier(_handle):
            calls[0] += 1
            stream.synchronize()
            dist.barrier()

        plan.allgather_multi(G, mapping, me, send, bases, barrier, stream)
        stream.synchronize()
        assert calls[0] == plan.num_steps + 1
        want, _ = oracle.allgather(algo, P, m, host_send)
        got = recv.cpu().numpy().reshape(len(mine), P * m)
        for li, r in enumerate(mine):
            assert np.array_equal(got[li], want[r]), (algo, P, m, "rank", r)
        dist.barrier()  # the other process may still be reading through its mapping
        while opened:
            sp.ipc_close(opened.pop())
        dist.barrier()  # nobody frees an allocation that is still mapped elsewhere
        del recv, send
    # the same through the package's torch.distributed wrapper, two collectives in a row
    for P, m in ((21, 528), (32, 8192)):
        ag = sp.multi.MultiDeviceAllgather(P, m, mapping=mapping, device=dev)
        for seed in (1, 2):
            host_send = si.send_blocks(P, m, seed=70 + seed)
            send = torch.from_numpy(np.ascontiguousarray(host_send[ag.ranks]).reshape(-1)).to(dev)
            ag.recv.fill_(si.SENTINEL)
            torch.cuda.synchronize()
            dist.barrier()  # nobody stores into a buffer that is still being filled
            with torch.cuda.stream(stream):
                got = ag.allgather(send)
            stream.synchronize()
            want, _ = oracle.allgather(sp.ALGO_SPARBIT, P, m, host_send)
            got = got.cpu().numpy()[: ag.n_local * P * m].reshape(ag.n_local, P * m)
            for li, r in enumerate(ag.ranks):
                assert np.array_equal(got[li], want[r]), ("wrapper", P, m, "rank", r)
        assert ag.barrier_calls == 2 * (ag.plan.num_steps + 1)
        ag.close()
    dist.destroy_process_group()
    print("multi-device worker ok", me)


if __name__ == "__main__":
    main()

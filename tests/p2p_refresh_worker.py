"""Child process of the peer-to-peer refresh test: a one-rank NCCL group with
torch symmetric memory, the refresh with exchange="p2p" against
exchange="allgather".  Prints OK, or SKIP and the reason when symmetric memory
is not usable on this machine."""

import os
import sys

import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def main():
    import torch.distributed as td
    from paper_2608_20818_b200 import binding as B
    from paper_2608_20818_b200 import sharded as S
    from tests import util as U

    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(29600 + os.getpid() % 300), RANK="0", WORLD_SIZE="1")
    torch.cuda.set_device(0)
    try:
        td.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", 0))
        probe = S.SymmetricSendBuffers(1024, torch.device("cuda", 0))
        probe.barrier(0)
        torch.cuda.synchronize()
        del probe
    except Exception as e:                           # no NCCL group or no symmetric memory on this machine
        print("SKIP", type(e).__name__, str(e)[:200])
        return
    shapes = [(512, 1024), (1024, 512), (1024, 2560), (300, 520)]
    W, G, M = U.make_inputs(shapes, 31, "bf16", grad_std=1e-3, mom_std=1e-3)
    out = {}
    for mode in ("allgather", "p2p"):
        opt = B.PeriodicRowwiseMuon(shapes, 1, 0.95, True, 5e-3, 0.01)
        P = [w.cuda() for w in W]
        Gd = [g.cuda() for g in G]
        Md = [m.cuda() for m in M]
        buffers = {}
        backend = S.CudaRefreshBackend(opt, 0.95, True)
        try:
            if mode == "p2p":
                # force the symmetric-memory path although the group has one rank
                symm = S.SymmetricSendBuffers(4 << 20, torch.device("cuda", 0))
                assert len(symm.ptrs(0)) == 1 and symm.ptrs(0)[0] == symm.tensors[0].data_ptr()
                buffers.update(key=("p2p", None), symm=symm, send=symm.tensors)
                plan = B.prm_bucket_plan(shapes, 1, 4 << 20)
                buffers["key"] = ("p2p", max(plan[2]), 1, "cuda:0")
        except Exception as e:                       # symmetric memory not available here
            print("SKIP", type(e).__name__, str(e)[:200])
            td.destroy_process_group()
            return
        for _ in range(2):
            S.bucketed_refresh_step(shapes, P, Gd, Md, backend, bucket_bytes=4 << 20, buffers=buffers, exchange=mode)
        torch.cuda.synchronize()
        assert opt.status() == B.PRM_OK
        out[mode] = ([p.cpu() for p in P], [m.cpu() for m in Md])
        opt.close()
    for a, b in zip(out["allgather"][0] + out["allgather"][1], out["p2p"][0] + out["p2p"][1]):
        assert torch.equal(a, b)
    td.destroy_process_group()
    print("OK")


if __name__ == "__main__":
    main()

"""The exchange step of the data-parallel form on CPU (gloo, world size 2): every rank ends with the mean of the
ranks' weight gradients, which is what the oracle's parameter server computes from the nodes' gradients."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _node_grads(rank):
    r = np.random.default_rng(100 + rank)
    return [r.normal(size=s).astype(np.float32) for s in ((6, 5), (4, 3, 3, 3), (7,))]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    sys.path.insert(0, ROOT)
    from paper_2004_04729_b200.binding import average_weight_gradients
    dist.init_process_group("gloo", rank=rank, world_size=world)
    grads = [torch.from_numpy(g.copy()) for g in _node_grads(rank)]
    average_weight_gradients(grads + [None])
    out.put((rank, [g.numpy().copy() for g in grads]))
    dist.barrier()
    dist.destroy_process_group()


def test_every_rank_ends_with_the_parameter_servers_average():
    import oracle
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 31500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = dict(out.get(timeout=180) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    per_node = [_node_grads(r) for r in range(2)]
    for i in range(3):
        want = oracle.parameter_server_average([per_node[0][i], per_node[1][i]])
        for rank in range(2):
            np.testing.assert_allclose(got[rank][i], want, rtol=0, atol=1e-7)
            assert got[rank][i].shape == per_node[0][i].shape


def test_without_a_process_group_nothing_happens():
    sys.path.insert(0, ROOT)
    from paper_2004_04729_b200.binding import average_weight_gradients
    g = torch.ones(3)
    average_weight_gradients([g])
    assert torch.equal(g, torch.ones(3))

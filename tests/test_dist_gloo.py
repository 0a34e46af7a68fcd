"""World-size-2 run of the multi-GPU plumbing on CPU (gloo): sharding and scalar reduces."""
import os
import socket

import numpy as np
import torch.multiprocessing as mp

import oracle
from paper_2202_07471_b200 import workloads as W


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    from paper_2202_07471_b200 import dist as D
    r, w, _ = D.init_from_env(world, backend="gloo")
    D.barrier()
    mx = D.max_over_ranks(10.0 + r)
    sm = D.sum_over_ranks(1.0 + r)
    shapes = [(8, 4, 3, 3), (5, 6, 1, 1), (1, 3, 3, 3)]
    pieces = D.shard_channels(shapes, r, w)
    # each rank quantizes its pieces with the CPU checker; the union must equal the unsplit result
    outs = []
    for layer, c0, n in pieces:
        wfull = W.random_layer(shapes[layer], seed=layer)
        res = oracle.quantize_layer(wfull[c0:c0 + n], bits=4)
        outs.append((layer, c0, n, res.codes.tobytes(), res.scales.tobytes()))
    q.put((r, mx, sm, outs))
    D.finish()


def test_two_ranks_shard_without_exchange():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = [q.get(timeout=120) for _ in range(world)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    shapes = [(8, 4, 3, 3), (5, 6, 1, 1), (1, 3, 3, 3)]
    full = [oracle.quantize_layer(W.random_layer(s, seed=i), bits=4) for i, s in enumerate(shapes)]
    covered = [np.zeros(s[0], dtype=int) for s in shapes]
    for r, mx, sm, outs in got:
        assert mx == 11.0 and sm == 3.0
        for layer, c0, n, codes, scales in outs:
            covered[layer][c0:c0 + n] += 1
            assert codes == full[layer].codes[c0:c0 + n].tobytes()
            assert scales == full[layer].scales[c0:c0 + n].tobytes()
    assert all((c == 1).all() for c in covered)

"""World-size-2 check of the data-parallel plumbing on CPU (gloo): batch sharding and the gradient
average of Algorithm 1.  Each rank computes its batch's gradient with the CPU oracle (this is a test, so
the oracle may stand in for the GPU step), the ranks all-reduce through the same helper bench.py uses,
and the result must equal the oracle's average of the two workers' gradients."""
import os
import socket
import sys

import numpy as np
import pytest

torch = pytest.importorskip("torch")
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import oracle
    import workloads as wl
    from paper_2506_20818_b200.dp import batch_for, sync_gradients

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    g, X, params, pos, cfg = wl.make_config("c2_chunglu_sage2", scale=0.005)
    dims = [128, 64, 32]
    params = wl.glorot_params("sage", dims, 3, 0.05)
    B = 256
    nb = len(pos[0]) // B
    step = 5
    b = batch_for(step, rank, world, nb)
    u, v = pos[0][b * B:(b + 1) * B], pos[1][b * B:(b + 1) * B]
    ns, nd, _ = oracle.sample_negatives(g.n, g.rowptr, g.col, u, 7, step, 1, edge_index_base=b * B)
    grads = torch.from_numpy(oracle.train_step(g, X, params, "sage", dims, u, v, ns, nd)["grads"].copy())
    mine = grads.clone()
    scale = sync_gradients(grads, world, dist)
    np.save(os.path.join(out_dir, f"avg_{rank}.npy"), (grads * scale).numpy())
    np.save(os.path.join(out_dir, f"own_{rank}.npy"), mine.numpy())
    np.save(os.path.join(out_dir, f"batch_{rank}.npy"), np.array([b]))
    dist.destroy_process_group()


def test_two_rank_gradient_average(tmp_path):
    import torch.multiprocessing as mp
    import oracle
    port = _free_port()
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    avg = [np.load(tmp_path / f"avg_{r}.npy") for r in range(2)]
    own = [np.load(tmp_path / f"own_{r}.npy") for r in range(2)]
    batches = [int(np.load(tmp_path / f"batch_{r}.npy")[0]) for r in range(2)]
    assert batches[0] != batches[1] and batches == [10, 11]  # step 5, two ranks: batches 10 and 11
    assert np.array_equal(avg[0], avg[1])                    # every rank holds the same averaged gradient
    assert np.allclose(avg[0], oracle.average_gradients(own), rtol=1e-14, atol=0)
    assert not np.allclose(own[0], own[1])


def test_batch_sharding_covers_every_batch_once():
    sys.path.insert(0, ROOT)
    from paper_2506_20818_b200.dp import batch_for
    for world in (1, 2, 4, 8):
        nb = 30
        seen = [batch_for(s, r, world, nb) for s in range(nb) for r in range(world)]
        counts = np.bincount(seen, minlength=nb)
        assert counts.min() == counts.max() == world  # nb steps of `world` ranks visit each batch `world` times
        assert len({batch_for(3, r, world, nb) for r in range(world)}) == world

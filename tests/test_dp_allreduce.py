"""The one exchange step of a data-parallel layer step: dS summed over the ranks in one flat
bucket (the scale gradient of Eq. 2 is a sum over tokens, and the ranks split the tokens).
Two gloo ranks on CPU; the expected values come from the oracle on the whole batch."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _case():
    sys.path.insert(0, ROOT)
    import oracle
    from paper_2305_14152_b200 import synth
    layers = []
    for i, (N, K, bits, g) in enumerate([(24, 64, 4, 0), (16, 128, 3, 32), (40, 64, 3, 64)]):
        d = synth.custom(50 + i, N, K, 12, bits, g)
        codes, zeros, scales = oracle.quantize_rtn(d["W"], bits, g)
        layers.append((d, oracle.pack(codes, bits), zeros, bits, g))
    return oracle, layers


def _worker(rank, world, port, q):
    oracle, layers = _case()
    from paper_2305_14152_b200 import dp
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # this rank's tokens: rows rank::world of the batch
    grads = []
    for d, packed, zeros, bits, g in layers:
        rows = np.arange(rank, d["X"].shape[0], world)
        ds = oracle.bwd_ds(np.ascontiguousarray(d["X"][rows]), np.ascontiguousarray(d["dY"][rows]), packed, zeros,
                           bits, g)
        grads.append(torch.from_numpy(ds.astype(np.float32)))
    # route 1: separate tensors, copied through a bucket
    a = [t.clone() for t in grads]
    dp.allreduce_scale_grads(a)
    # route 2: the tensors are views of the bucket already (what the kernels write into)
    bucket, views = dp.bucket_views(grads)
    for v, t in zip(views, grads):
        v.copy_(t)
    dp.allreduce_scale_grads(views, bucket=bucket)
    # route 3: average
    c = [t.clone() for t in grads]
    dp.allreduce_scale_grads(c, average=True)
    q.put((rank, [t.numpy() for t in a], [v.numpy().copy() for v in views], [t.numpy() for t in c],
           [int(v.data_ptr() - bucket.data_ptr()) for v in views]))
    dist.barrier()
    dist.destroy_process_group()


def test_scale_gradients_sum_over_two_ranks():
    oracle, layers = _case()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = {}
    for _ in range(2):
        r = q.get(timeout=180)
        got[r[0]] = r[1:]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    whole = [oracle.bwd_ds(d["X"], d["dY"], packed, zeros, bits, g) for d, packed, zeros, bits, g in layers]
    for rank in (0, 1):
        summed, in_bucket, averaged, offsets = got[rank]
        for ref, s, b, avg in zip(whole, summed, in_bucket, averaged):
            tol = 1e-5 * np.abs(ref).max()       # two fp32 partial sums against one fp64 sum
            assert s.shape == ref.shape and np.abs(s - ref).max() <= tol
            assert np.array_equal(s, b)
            assert np.abs(avg - ref / 2).max() <= tol
        assert all(o % 256 == 0 for o in offsets)
    assert all(np.array_equal(x, y) for x, y in zip(got[0][0], got[1][0]))   # ranks agree bit for bit


def test_without_a_process_group_nothing_changes():
    sys.path.insert(0, ROOT)
    from paper_2305_14152_b200 import dp
    g = [torch.arange(6, dtype=torch.float32).view(2, 3)]
    assert dp.allreduce_scale_grads(g)[0] is g[0]
    bucket, views = dp.bucket_views([torch.zeros(5), torch.zeros(70)])
    assert bucket.numel() == 64 + 128 and views[1].shape == (70,)

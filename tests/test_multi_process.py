"""Host-side logic of the N > 1 path on CPU (gloo, world size 2): the batch is sharded over the
ranks with no data-path collective, each rank's shard gives exactly the rows of the full
result (sequences are independent), the parameter gradients add up across ranks, and the
step time reported is the maximum over ranks.  The second test covers the exchange a data-parallel
trainer adds: the five parameter gradients summed over the ranks by one all-reduce of the bucket
they live in."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import ssm_oracle as O
from paper_2502_20168_b200 import inputs as I

W = I.Workload("mp", B=5, T=12, H=8, P=8, p_done=0.2, seed=3)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    d = I.draw_layer(W)
    lo, hi = I.shard_batch(W.B, rank, world)
    args = (d["Lambda"], d["Delta"], d["Bc"], d["Cc"], d["D"])
    y, _, _ = O.ssm_layer_fwd(*args, d["u"][lo:hi], d["done"][lo:hi], None)
    g = O.ssm_layer_bwd(*args, d["u"][lo:hi], d["done"][lo:hi], None, d["gy"][lo:hi])
    dC = torch.from_numpy(np.stack([g["dC"].real, g["dC"].imag]))
    dist.all_reduce(dC)                                    # what a data-parallel trainer would add
    t = torch.tensor([1.0 + rank], dtype=torch.float64)    # this rank's step time
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    out.put((rank, lo, hi, y, dC.numpy(), float(t)))
    dist.barrier()
    dist.destroy_process_group()


def _bucket_rank_main(rank, world, port, out):
    import types
    from paper_2502_20168_b200 import harness
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    d = I.draw_layer(W)
    lo, hi = I.shard_batch(W.B, rank, world)
    g = O.ssm_layer_bwd(d["Lambda"], d["Delta"], d["Bc"], d["Cc"], d["D"], d["u"][lo:hi], d["done"][lo:hi], None,
                        d["gy"][lo:hi])
    bucket, views = harness.grad_bucket(W.P, W.H, "cpu")
    names = ("dLambda", "dDelta", "dB", "dC", "dD")
    for name, v in zip(names, views):          # this rank's gradients, where the layer's backward would put them
        v.copy_(torch.from_numpy(np.ascontiguousarray(g[name])).to(v.dtype))
    buf = types.SimpleNamespace(grad_bucket=bucket)
    work = harness.allreduce_param_grads(buf, async_op=True)
    work.wait()
    out.put((rank, {name: v.numpy().copy() for name, v in zip(names, views)}))
    dist.barrier()
    dist.destroy_process_group()


def _exchange_order_rank_main(rank, world, port, out):
    """Three steps of a training loop's gradient exchange: backward writes the bucket, start(), the next forward
    runs, finish() before the next backward."""
    import types
    from paper_2502_20168_b200 import harness
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    bucket, _ = harness.grad_bucket(W.P, W.H, "cpu")
    x = harness.GradExchange(types.SimpleNamespace(grad_bucket=bucket))
    sums, refused = [], False
    for step in range(3):
        x.finish()                                   # before the backward pass rewrites the bucket
        bucket.fill_(float(10 * step + rank + 1))    # "backward": this rank's gradients of this step
        x.start()
        if step == 1:
            try:
                x.start()                            # a rewrite + restart without finish() must be refused
            except RuntimeError:
                refused = True
        # (the next step's forward pass would run here, under the exchange)
        x.finish()
        sums.append(float(bucket[0]))
        assert torch.all(bucket == bucket[0])
    out.put((rank, sums, refused, x.started, x.finished))
    dist.barrier()
    dist.destroy_process_group()


def test_gradient_exchange_is_finished_before_the_bucket_is_rewritten():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_exchange_order_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = [q.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, sums, refused, started, finished in got:
        assert sums == [3.0, 23.0, 43.0]             # (10 s + 1) + (10 s + 2) per step s, never a mix of two steps
        assert refused and started == finished == 3


def test_parameter_gradients_summed_over_two_ranks_by_one_bucket_allreduce():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_bucket_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = [q.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    d = I.draw_layer(W)
    g = O.ssm_layer_bwd(d["Lambda"], d["Delta"], d["Bc"], d["Cc"], d["D"], d["u"], d["done"], None, d["gy"])
    for rank, grads in got:
        for name, v in grads.items():          # fp32 bucket against the float64 full-batch gradients
            ref = g[name]
            assert v.shape == ref.shape, name
            assert np.max(np.abs(v - ref) / (1.0 + np.abs(ref))) < 1e-5, (rank, name)


def test_batch_sharding_over_two_ranks():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = [q.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    d = I.draw_layer(W)
    args = (d["Lambda"], d["Delta"], d["Bc"], d["Cc"], d["D"])
    y, _, _ = O.ssm_layer_fwd(*args, d["u"], d["done"], None)
    g = O.ssm_layer_bwd(*args, d["u"], d["done"], None, d["gy"])
    covered = np.zeros(W.B, bool)
    for rank, lo, hi, yr, dC, t in got:
        assert np.allclose(yr, y[lo:hi], atol=1e-12)
        assert not covered[lo:hi].any()
        covered[lo:hi] = True
        assert np.allclose(dC[0] + 1j * dC[1], g["dC"], atol=1e-10)
        assert t == 2.0
    assert covered.all()

"""The data-parallel form of the layer-wise regression step (Section 3.1, Eq. (w_b)) on two CPU processes (gloo): each
rank takes the checker's gradients of its shard of the mini-batch with the mini-batch's constant, one sum-all-reduce
carries dW, db and the loss, and every rank applies the same update.  The result is the single-process step on the whole
mini-batch.  (The arithmetic each GPU rank runs is dr_regress_shard_grads; its parity with these shard sums is a GPU test.)"""
import os
import socket
import sys

import numpy as np
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SHAPE = dict(B=6, H=8, Cin=5, Cout=7, k=3, s=1, p=1)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _problem():
    rng = np.random.default_rng(3)
    q = SHAPE
    x = rng.normal(size=(q["B"], q["H"], q["H"], q["Cin"]))
    yt = np.abs(rng.normal(size=(q["B"], q["H"], q["H"], q["Cout"])))
    w = rng.normal(size=(q["Cout"], q["k"], q["k"], q["Cin"])) * 0.2
    b = rng.normal(size=q["Cout"]) * 0.1
    return x, yt, w, b


def _worker(rank, world, port, out):
    import torch
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import oracle.finetune as F
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    x, yt, w, b = _problem()
    q = SHAPE
    bounds = [0, 4, q["B"]]                                  # uneven shards: 4 + 2 images
    lo, hi = bounds[rank], bounds[rank + 1]
    dw, db, loss = F.shard_gradients(x[lo:hi], yt[lo:hi], w, b, q["B"], q["s"], q["p"])
    flat = torch.from_numpy(np.concatenate([dw.ravel(), db.ravel(), [loss]]))
    dist.all_reduce(flat, op=dist.ReduceOp.SUM)              # the step's one collective: Cout*k*k*Cin + Cout + 1 values
    g = flat.numpy()
    dw_all, db_all, loss_all = g[:dw.size].reshape(dw.shape), g[dw.size:dw.size + db.size], float(g[-1])
    w2, _ = F.sgd_update(w, np.zeros_like(w), dw_all, 0.05, 0.9, 1e-4)
    b2, _ = F.sgd_update(b, np.zeros_like(b), db_all, 0.05, 0.9, 0.0)
    out.put((rank, w2.tolist(), b2.tolist(), loss_all))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_step_equals_the_whole_mini_batch_step():
    sys.path.insert(0, ROOT)
    import oracle.finetune as F
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=180) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    x, yt, w, b = _problem()
    q = SHAPE
    w_ref, b_ref, _, _, loss_ref, _, _ = F.regression_step(x, yt, w, b, np.zeros_like(w), np.zeros_like(b), 0.05, 0.9, 1e-4, q["s"], q["p"])
    for rank, w2, b2, loss in res:
        assert np.allclose(np.array(w2), w_ref, rtol=0, atol=1e-12)
        assert np.allclose(np.array(b2), b_ref, rtol=0, atol=1e-12)
        assert abs(loss - loss_ref) < 1e-12
    assert res[0][1] == res[1][1]                            # both ranks hold the same updated filters, bit for bit

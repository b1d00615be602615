"""The parameter-sharded Adam step on CPU: gloo ranks run the host logic of ShardedLowPrecisionAdam (shard bounds,
offsets, step-indexed seeds, gradient reduce-scatter, in-place all-gather of the codes) with the oracle standing in
for the device kernel, which needs a GPU.  After every step each rank must hold exactly the codes of one unsharded
call, and the master shards must be the slices of the unsharded master weights."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2504_20634_b200 import sharding
from paper_2504_20634_b200.sharded_optimizer import ShardedLowPrecisionAdam

HYPER = dict(lr=1e-3, betas=(0.9, 0.99), eps=1e-8)


def oracle_step(master_w, grad, m, v, fmt, variant, k_bits, seed, offset, lr, beta1, beta2, eps, step, out=None):
    """Same signature as the binding's fbsr_adam_update, on CPU tensors."""
    from oracle import capi
    codes = capi.adam_update(master_w.numpy(), grad.numpy(), m.numpy(), v.numpy(), fmt, variant, k_bits, seed, offset,
                             lr, beta1, beta2, eps, step)
    out.copy_(torch.from_numpy(codes.view(np.int16)).view(torch.uint16) if codes.dtype == np.uint16 else torch.from_numpy(codes))
    return out


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _inputs(n_total, world, steps):
    g = torch.Generator().manual_seed(77)
    w0 = torch.randn(n_total, generator=g) * 0.02
    # per-rank gradients of the full vector; their sum is what the update must see.  Small integer multiples of
    # 2^-20, so that the sum is exact in binary32 whatever order the collective adds them in
    grads = [[torch.randint(-2000, 2001, (n_total,), generator=g).float() * 2.0 ** -20 for _ in range(world)]
             for _ in range(steps)]
    return w0, grads


def _worker(rank, world, port, n_total, fmt, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from oracle import capi
        steps = 3
        w0, grads = _inputs(n_total, world, steps)
        dt = torch.uint16 if fmt in ("bf16", "fp16") else torch.uint8
        opt = ShardedLowPrecisionAdam(n_total, fmt=fmt, variant="src", k_bits=3, seed=40, device="cpu",
                                      step_fn=oracle_step, code_dtype=dt, **HYPER)
        opt.load_master(w0)
        # the unsharded run, on every rank (cheap): one call over the whole vector per step
        w, m, v = w0.numpy().copy(), np.zeros(n_total, np.float32), np.zeros(n_total, np.float32)
        ok = opt.shard_len % sharding.SHARD_ALIGN == 0 and opt.start == min(n_total, rank * opt.shard_len)
        buffers = set()
        for t in range(steps):
            if t == 1:
                # the gradients written straight into the optimizer's persistent buffer, the gather left in flight
                opt.grad_buffer().copy_(grads[t][rank])
                shard_grad = opt.reduce_scatter_grad()
                assert opt.step(shard_grad, wait=False) is None
                lp = opt.lp
            else:
                shard_grad = opt.reduce_scatter_grad(grads[t][rank])
                lp = opt.step(shard_grad)
            buffers.add((opt._grad_padded.data_ptr(), opt._grad_shard.data_ptr(), opt.lp_padded.data_ptr()))
            ok = ok and bool((opt._grad_padded[n_total:] == 0).all())
            acc = grads[t][0].clone()
            for r in range(1, world):
                acc += grads[t][r]
            whole = capi.adam_update(w, acc.numpy(), m, v, fmt, "src", 3, 40 + t + 1, 0, HYPER["lr"], 0.9, 0.99, 1e-8, t + 1)
            got = lp.view(torch.int16).numpy().view(np.uint16) if dt == torch.uint16 else lp.numpy()
            ok = ok and np.array_equal(got, whole)
            ok = ok and np.array_equal(opt.master.numpy(), w[opt.start:opt.end]) and np.array_equal(opt.m.numpy(), m[opt.start:opt.end])
        ok = ok and len(buffers) == 1          # nothing is reallocated from step to step
        with open(os.path.join(out_dir, "result%d" % rank), "w") as fh:
            fh.write("ok" if ok else "mismatch")
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world,fmt,n_total", [(2, "bf16", 2 * 15360 + 777), (3, "e4m3", 15360 + 5), (2, "b8p4", 100)])
def test_sharded_step_equals_unsharded(tmp_path, world, fmt, n_total):
    mp.spawn(_worker, args=(world, _free_port(), n_total, fmt, str(tmp_path)), nprocs=world, join=True)
    for r in range(world):
        assert open(tmp_path / ("result%d" % r)).read() == "ok"


def test_single_process_without_a_group():
    n = 5000
    w0, grads = _inputs(n, 1, 2)
    opt = ShardedLowPrecisionAdam(n, fmt="fp16", variant="srf", k_bits=4, seed=3, device="cpu", step_fn=oracle_step,
                                  code_dtype=torch.uint16, **HYPER)
    assert (opt.start, opt.end, opt.world) == (0, n, 1)
    opt.load_master(w0)
    from oracle import capi
    w, m, v = w0.numpy().copy(), np.zeros(n, np.float32), np.zeros(n, np.float32)
    for t in range(2):
        lp = opt.step(opt.reduce_scatter_grad(grads[t][0]))
        whole = capi.adam_update(w, grads[t][0].numpy(), m, v, "fp16", "srf", 4, 3 + t + 1, 0, HYPER["lr"], 0.9, 0.99, 1e-8, t + 1)
        assert np.array_equal(lp.view(torch.int16).numpy().view(np.uint16), whole)
    with pytest.raises(ValueError):
        opt.step(torch.zeros(n - 1))

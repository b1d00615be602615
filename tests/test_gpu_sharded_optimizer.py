"""ShardedLowPrecisionAdam on one GPU: the default step function is the library's fused kernel, the collective
runs through NCCL (a group of one rank; more ranks need more GPUs and are covered on CPU with gloo)."""
import socket

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_one_rank_nccl_group_equals_direct_calls():
    import torch.distributed as dist
    import paper_2504_20634_b200 as fbsr
    from paper_2504_20634_b200.sharded_optimizer import ShardedLowPrecisionAdam
    from oracle import capi
    import gpu_util as gu
    started = False
    if not dist.is_initialized():
        dist.init_process_group("nccl", init_method="tcp://127.0.0.1:%d" % _free_port(), rank=0, world_size=1,
                                device_id=torch.device("cuda", 0))
        started = True
    try:
        n = 3 * 15360 + 123
        g = torch.Generator(device="cuda").manual_seed(5)
        w0 = torch.randn(n, device="cuda", generator=g) * 0.02
        opt = ShardedLowPrecisionAdam(n, fmt="bf16", variant="srf", k_bits=4, seed=10, lr=1e-3, betas=(0.9, 0.99), eps=1e-8)
        opt.load_master(w0)
        w, m, v = w0.clone(), torch.zeros(n, device="cuda"), torch.zeros(n, device="cuda")
        wh, mh, vh = w0.cpu().numpy().copy(), np.zeros(n, np.float32), np.zeros(n, np.float32)
        for t in range(1, 4):
            grad = torch.randn(n, device="cuda", generator=g) * 1e-3
            lp = opt.step(opt.reduce_scatter_grad(grad))
            direct = fbsr.fbsr_adam_update(w, grad, m, v, "bf16", "srf", 4, 10 + t, 0, 1e-3, 0.9, 0.99, 1e-8, t)
            assert torch.equal(lp, direct) and torch.equal(opt.master, w) and torch.equal(opt.v, v)
            expect = capi.adam_update(wh, grad.cpu().numpy(), mh, vh, "bf16", "srf", 4, 10 + t, 0, 1e-3, 0.9, 0.99, 1e-8, t)
            gu.assert_codes_equal(lp, expect, "step %d" % t)
        # the gradients written straight into the optimizer's persistent buffer, the gather left to be waited for later:
        # same result, and a step takes no memory from the allocator
        for t in range(4, 7):
            grad = torch.randn(n, device="cuda", generator=g) * 1e-3
            opt.grad_buffer().copy_(grad)
            torch.cuda.synchronize()
            allocated = torch.cuda.memory_allocated()
            assert opt.step(opt.reduce_scatter_grad(), wait=False) is None
            torch.cuda.synchronize()
            assert torch.cuda.memory_allocated() == allocated
            direct = fbsr.fbsr_adam_update(w, grad, m, v, "bf16", "srf", 4, 10 + t, 0, 1e-3, 0.9, 0.99, 1e-8, t)
            assert torch.equal(opt.lp, direct) and torch.equal(opt.master, w) and torch.equal(opt.m, m)
        # the collective itself, as step() issues it for more than one rank: in place, on bytes
        own = opt.lp_padded[: opt.shard_len]
        before = opt.lp_padded.clone()
        dist.all_gather_into_tensor(opt.lp_padded.view(torch.uint8), own.view(torch.uint8))
        torch.cuda.synchronize()
        assert torch.equal(opt.lp_padded, before)
    finally:
        if started:
            dist.destroy_process_group()

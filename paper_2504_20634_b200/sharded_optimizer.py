"""Parameter-sharded fused Adam step with a low-precision all-gather (one process per GPU).

Every rank holds the whole low-precision copy of a flat parameter vector (what the forward and backward
passes read) but the binary32 master weights and Adam moments of its own shard only.  One step is

    1. (optional) reduce-scatter of the binary32 gradients, so that each rank gets the summed gradient
       of its shard; the gradients live in a persistent padded buffer, so the step allocates nothing;
    2. the fused update of the shard: master weights and moments in place, and the stochastically rounded
       weights written straight into this rank's slice of the full low-precision buffer (the last line
       of Algorithm 1: the SR write lands in the buffer that the collective sends, no staging copy);
    3. an in-place all-gather of that buffer over the process group (NCCL over NVLink on GPUs), issued
       asynchronously so that it overlaps what the caller enqueues next.

Draws are keyed by the global element index (``offset`` = start of the shard) and the seed of step t is
``seed + t``, so the gathered codes are bit-identical to one unsharded call on one GPU.  The only data
that crosses ranks is the gradient reduce-scatter and the code all-gather; there is no other exchange.

Host-side logic only: the arithmetic is the library's fused kernel (``fbsr_adam_update``).  ``step_fn``
exists so that the plumbing can be exercised where no GPU is present; it must have that function's
signature.
"""
import torch

from . import sharding


def _dist(group):
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        return dist, dist.get_rank(group), dist.get_world_size(group)
    return None, 0, 1


class ShardedLowPrecisionAdam:
    def __init__(self, n_total, fmt="bf16", variant="srf", k_bits=4, seed=0, lr=1e-4, betas=(0.9, 0.999), eps=1e-8,
                 device="cuda", group=None, step_fn=None, code_dtype=None):
        if n_total < 0:
            raise ValueError("n_total must be non-negative")
        self.dist, self.rank, self.world = _dist(group)
        self.group = group
        self.n_total, self.fmt, self.variant, self.k_bits = n_total, fmt, variant, k_bits
        self.seed, self.lr, self.betas, self.eps = seed, lr, betas, eps
        self.device = torch.device(device)
        if step_fn is None:
            from . import binding
            step_fn = binding.fbsr_adam_update
            code_dtype = binding.CODE_DTYPE[fmt]
        elif code_dtype is None:
            raise ValueError("code_dtype must be given with a custom step_fn")
        self.step_fn = step_fn
        # equal shard lengths (the collective needs them), on the grid that keeps every k on the tiled kernels
        align = sharding.SHARD_ALIGN
        per_rank = -(-n_total // self.world)
        self.shard_len = max(align, -(-per_rank // align) * align)
        self.start = min(n_total, self.rank * self.shard_len)
        self.end = min(n_total, self.start + self.shard_len)
        self.n_own = self.end - self.start
        f32 = dict(dtype=torch.float32, device=self.device)
        self.master = torch.zeros(self.n_own, **f32)
        self.m = torch.zeros(self.n_own, **f32)
        self.v = torch.zeros(self.n_own, **f32)
        self.lp_padded = torch.zeros(self.world * self.shard_len, dtype=code_dtype, device=self.device)
        self.step_count = 0
        self._gather = None                # handle of the all-gather in flight
        self._grad_padded = None           # made on first use by grad_buffer()
        self._grad_shard = None

    @property
    def lp(self):
        """The full low-precision parameter vector (n_total codes), valid on every rank after step(); waits for
        the all-gather in flight."""
        self.wait_gather()
        return self.lp_padded[: self.n_total]

    def _own_slice(self):
        a = self.rank * self.shard_len
        return self.lp_padded[a: a + self.shard_len]

    def load_master(self, full_or_shard):
        """Set the master weights from the full vector (every rank takes its shard) or from the shard itself."""
        src = full_or_shard
        if src.numel() == self.n_total and self.n_total != self.n_own:
            src = src[self.start: self.end]
        if src.numel() != self.n_own:
            raise ValueError("expected %d or %d elements" % (self.n_total, self.n_own))
        self.master.copy_(src)

    def grad_buffer(self):
        """The persistent full-length gradient buffer (n_total binary32 values) that the backward pass may write
        into directly; it is the front of a world x shard_len buffer whose tail stays zero, so that
        reduce_scatter_grad() needs neither an allocation nor a padding copy."""
        if self._grad_padded is None:
            self._grad_padded = torch.zeros(self.world * self.shard_len, dtype=torch.float32, device=self.device)
            self._grad_shard = torch.empty(self.shard_len, dtype=torch.float32, device=self.device)
        return self._grad_padded[: self.n_total]

    def reduce_scatter_grad(self, full_grad=None):
        """Sum the ranks' gradients of the full vector and return this rank's shard of the sum.  Without an
        argument the gradients are taken from grad_buffer() (no copy); a tensor given here is first copied into
        that buffer.  Nothing is allocated after the first call."""
        buf = self.grad_buffer()
        if full_grad is not None and full_grad.data_ptr() != buf.data_ptr():
            if full_grad.numel() != self.n_total:
                raise ValueError("full_grad must have n_total elements")
            if self.world == 1:
                return full_grad[self.start: self.end]
            buf.copy_(full_grad)
        if self.world == 1:
            return buf[self.start: self.end]
        self.dist.reduce_scatter_tensor(self._grad_shard, self._grad_padded, group=self.group)
        return self._grad_shard[: self.n_own]

    def step(self, grad_shard, wait=True):
        """One fused step on this rank's shard, then the all-gather of the codes, issued asynchronously (on the
        collective library's own stream under NCCL) so that whatever the caller enqueues next overlaps it.
        With wait=True (default) the current stream waits for the gather before this returns the full code vector;
        with wait=False the caller goes on and `lp` (or wait_gather()) does the waiting when the codes are needed."""
        if grad_shard.numel() != self.n_own:
            raise ValueError("grad_shard must have %d elements" % self.n_own)
        self.wait_gather()                 # the previous gather must be done before its buffer is rewritten
        self.step_count += 1
        own = self._own_slice()
        if self.n_own:
            self.step_fn(self.master, grad_shard.contiguous(), self.m, self.v, self.fmt, self.variant, self.k_bits,
                         self.seed + self.step_count, self.start, self.lr, self.betas[0], self.betas[1], self.eps,
                         self.step_count, out=own[: self.n_own])
        if self.world > 1:
            # bytes, so that the collective never meets a dtype it has no name for; in place: this rank's
            # input is its own slice of the output
            self._gather = self.dist.all_gather_into_tensor(self.lp_padded.view(torch.uint8), own.view(torch.uint8),
                                                            group=self.group, async_op=True)
        if wait:
            return self.lp
        return None

    def wait_gather(self):
        """Make the current stream (the host, on CPU) wait for the pending all-gather, if any."""
        if self._gather is not None:
            self._gather.wait()
            self._gather = None
